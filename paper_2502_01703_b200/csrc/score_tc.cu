// Stage 3 on the tensor cores for every code width. 8- and 4-bit codes: tcgen05.mma kind::i8, int32 accumulators in
// TMEM (4-bit codes expanded to int8 on the way). 2- and 1-bit codes: the codes -2 .. 1 and the signs +-1 are exact
// e2m1 values, so they run on the block-scaled fp4 path (kind::mxf4 with every scale factor 2^0, 64 codes per
// instruction instead of 32, fp32 accumulation of integers no larger than 4 d: exact), at twice the int8 rate.
//
// Two CTAs on neighbouring SMs form a pair (cta_group::2) and own a tile of 256 train rows (UMMA M), 128
// per CTA. For each checkpoint the pair streams the tile's codes and the validation codes K-block by
// K-block (128 operand bytes per row per block: 128 int8 codes or 256 e2m1 codes, 128-byte-swizzled K-major
// operands) and accumulates D[t, v] = sum_m q_t,m q_v,m for up to 512 validation vectors at once (two MMAs of
// N <= 256 per K step); each CTA stages only half of the validation rows of every MMA, which halves what an SM
// pulls from L2. After the last K block of a checkpoint the epilogue warps of each CTA read their half of the
// accumulator (thread = train row), apply the per-vector multipliers (Eq. 6), form the per-task means and add
// eta_i * mean to the running per-task sums; after the last checkpoint they take the max over tasks.
// The N x V x C similarity tensor never exists in memory.
//
// 8-bit train codes go from global memory to the MMA operand buffer by TMA. 4-bit train codes arrive packed (TMA,
// no swizzle) in a staging ring; unpack warps (thread = train row = TMEM lane) sign-extend them to int8 and store
// them straight into tensor memory, from where the MMA takes its A operand: no shared-memory write, no swizzle, no
// proxy fence. The accumulator leaves 64 of the 512 TMEM columns free, enough for two 128-code blocks of A, so at
// the sub-byte widths a validation tile holds at most 448 vectors. 2- and 1-bit train codes: the block-scaled MMA
// also reads its scale factors from tensor memory (8 columns), which a 448-column accumulator and two A slots leave
// no room for, so the unpack warps (three or four groups of four, each thread a row) take the packed codes straight
// from global memory (32 or 64 bytes per row and K block, whole sectors, two blocks ahead in registers), expand
// them to e2m1 and write the row into the operand stage in shared memory in the swizzled layout a TMA load would
// have produced (a proxy fence and, from the peer CTA, a cluster-scope release per warp and block).
// Validation codes are expanded once per call into a workspace (they are a few MB and stay in L2). Inside a
// 128-code block the 4-bit unpackers place the codes in a fixed permutation, the same for both operands, which an
// inner product does not see; the e2m1 codes stay in order.
//
// One barrier per pipeline stage on the leader CTA collects everything the MMAs of that stage need (TMA
// bytes of both CTAs, and the unpack warps' arrivals); one tcgen05.commit releases the stage in both CTAs:
// the single MMA-issuing thread runs at the tensor pipe's own pace, so every other instruction it executes
// is lost tensor time.
//
// Warp roles (448 threads per CTA; 704 / 832 for 1- / 2-bit codes): warp 0 TMA producer, warp 1 MMA issuer (leader
// only; + TMEM allocation), warps 2-5 and 10-13 unpack (idle for 8-bit, where 2-5 form a second epilogue group),
// warps 6-9 epilogue; 2- and 1-bit codes add unpack warps 14-17 (and 18-21 at 2 bits) and behind them four more
// epilogue warps that take half of the accumulator's columns. All waits are bounded.
#include "qless_kernels.h"
#include "tc_common.cuh"

namespace qless {

namespace {

using namespace tc;

constexpr int TM = 128;                    // train rows per tile
constexpr int KB = 128;                    // codes (= unpacked bytes) per row per K block
constexpr int A_STAGE = TM * KB;           // 16 KiB
constexpr int MAX_STAGES = 8;
constexpr int NTHREADS = 448;
// 2- and 1-bit codes: NG groups of four unpack warps (2-5, 10-13, 14-17, ...) and, behind them, four more epilogue warps
__host__ __device__ constexpr int fp4_groups(int bits) { return bits == 1 ? 3 : 4; }
__host__ __device__ constexpr int fp4_threads(int bits) { return NTHREADS + 128 * (fp4_groups(bits) - 2) + 128; }
constexpr int TMAX = 8;                    // tasks held in registers by the epilogue
constexpr int A_TMEM_COL = 448;            // sub-byte widths: two 32-column slots of unpacked train codes

struct ScoreTcParams {
    int64_t N;
    int32_t V, C, T, d, bits;
    int32_t vpad;               // validation rows per tile, multiple of 16, <= 512
    int32_t n1, n2;             // MMA N of the two halves (n1 + n2 = vpad)
    int32_t nS, nP;             // pipeline depths: operand stages (A + B), packed staging
    int32_t epi_groups;         // 1 or 2 groups of four epilogue warps (2: each takes half of the columns)
    const uint8_t* train_codes; // packed train codes (read directly by the unpack warps of the 2- and 1-bit path)
    int64_t train_stride;       // bytes between checkpoints
    const float* train_mult;    // [C][N]
    const float* val_mult;      // [C][V]
    const float* eta_over_cnt;  // [C][T]
    const int32_t* task_off;    // [T+1]
    float* scores;
    float* per_task;
    int32_t* dots;              // raw integer dots [N][V] (C = 1) instead of scores
    unsigned int* timeout_word;
};

struct __align__(8) ScoreBars {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES];
    uint64_t p_full[MAX_STAGES], p_empty[MAX_STAGES], d_full, d_empty, drain;
    uint32_t tmem_base, abort_flag;
    int32_t task_off[65];
    __align__(16) float mv[512];
    float eta_s[TMAX];          // this checkpoint's eta_i / |task j|
    float comb[TM][6];          // per-task partial sums handed from the second epilogue group to the first
};

// 8 packed 4-bit codes -> two words of four int8 (low nibbles, high nibbles)
__device__ __forceinline__ void unpack4(uint32_t w, uint32_t& lo, uint32_t& hi)
{
    lo = __vsub4((w & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);
    hi = __vsub4(((w >> 4) & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);
}
// Position in a ring of n slots: slot index and the parity of its current use. Advanced by comparison, not by
// division: the role loops below run on single threads whose every instruction is on the critical path.
struct Ring {
    uint32_t slot = 0, parity = 0;
    __device__ __forceinline__ void next(uint32_t n) { if (++slot == n) { slot = 0; parity ^= 1u; } }
};

// 16 sign bits (bit set = negative) -> two words of eight e2m1 codes (+1 = 0x2, -1 = 0xA), code j of the sixteen in
// nibble j: the bits are spread into eight 2-bit byte selectors, and a byte permute looks each pair of codes up.
__device__ __forceinline__ uint32_t spread2_to_nibbles(uint32_t h)          // 2-bit field j of 16 bits -> nibble j
{
    uint32_t x = (h | (h << 8)) & 0x00FF00FFu;
    x = (x | (x << 4)) & 0x0F0F0F0Fu;
    return (x | (x << 2)) & 0x33333333u;
}
__device__ __forceinline__ void fp4_from_signs16(uint32_t h, uint32_t& lo, uint32_t& hi)
{
    const uint32_t sel = spread2_to_nibbles(h);
    lo = __byte_perm(0xAAA22A22u, 0u, sel);              // selector 0..3 -> 0x22, 0x2A, 0xA2, 0xAA
    hi = __byte_perm(0xAAA22A22u, 0u, sel >> 16);
}
// 16 two-bit codes (two's complement) -> two words of eight e2m1 codes: 00 -> 0, 01 -> +1 (0x2), 11 -> -1 (0xA), 10 -> -2 (0xC)
__device__ __forceinline__ uint32_t fp4_from_nibble_codes2(uint32_t y)     // nibbles 00 c1 c0
{
    const uint32_t c0 = (y & 0x11111111u) << 1, c1 = y & 0x22222222u;
    return c0 | (c1 << 2) | ((c1 & ~c0) << 1);
}
__device__ __forceinline__ void fp4_from_codes2(uint32_t w, uint32_t& lo, uint32_t& hi)
{
    lo = fp4_from_nibble_codes2(spread2_to_nibbles(w & 0xFFFFu));
    hi = fp4_from_nibble_codes2(spread2_to_nibbles(w >> 16));
}

template <int BITS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(BITS <= 2 ? fp4_threads(BITS) : NTHREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmap_train, const __grid_constant__ CUtensorMap tmap_val1,
                const __grid_constant__ CUtensorMap tmap_val2, const ScoreTcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);    // 1 KiB aligned, still a shared pointer
    const int bh1 = (p.n1 / 2) * KB, bh2 = (p.n2 / 2) * KB;      // bytes of this CTA's rows of the two MMA halves
    constexpr bool DIRECT = (BITS >= 8);                           // 8-bit codes and bf16 rows feed the MMA as stored
    constexpr bool FP4 = (BITS <= 2);                              // 2- and 1-bit codes run as e2m1 (kind::mxf4): 256 codes per K block
    constexpr int A_SMEM = (DIRECT || FP4) ? A_STAGE : 0;         // 4-bit codes keep A in tensor memory
    const int stage_bytes = A_SMEM + bh1 + bh2;                   // multiple of 1024
    constexpr int PROW = DIRECT ? 0 : (FP4 ? 32 : 16) * BITS;     // packed bytes of one row's K block
    constexpr int P_STAGE = (DIRECT || FP4) ? 0 : TM * PROW;      // packed staging bytes per stage (4-bit codes only)
    uint8_t* sS = smem;                                           // stage s: [A 16 KiB][B half 1][B half 2]
    uint8_t* sP = sS + (size_t)p.nS * stage_bytes;
    ScoreBars* bars = reinterpret_cast<ScoreBars*>(sP + (size_t)p.nP * P_STAGE);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int64_t pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int nkb = (BITS == 16) ? (2 * p.d) / KB : FP4 ? (p.d + 2 * KB - 1) / (2 * KB) : p.d / KB;      // K blocks of 128 operand bytes per row
    const int num_vt = (p.V + p.vpad - 1) / p.vpad;
    const int64_t num_tiles = (p.N + 2 * TM - 1) / (2 * TM);      // tiles of 256 train rows
    // int8: D = S32 (2), A = B = S8 (1); 16-bit baseline: D = F32 (1), A = B = BF16 (1)
    const uint32_t idesc1 = FP4 ? make_idesc_mxf4(2 * TM, p.n1) : make_idesc(BITS == 16 ? 1 : 2, 1, 1, 2 * TM, p.n1);
    const uint32_t idesc2 = FP4 ? make_idesc_mxf4(2 * TM, p.n2 > 0 ? p.n2 : 16) : make_idesc(BITS == 16 ? 1 : 2, 1, 1, 2 * TM, p.n2 > 0 ? p.n2 : 16);

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) {
            // leader's full[s]: the producer's expect_tx arrival (+ one arrival per unpack warp of both CTAs)
            // (8-bit codes and bf16 rows: one barrier per PAIR of stages, at the even slot, collects both stages' arrivals,
            // so that the MMA-issuing thread waits once per 16 MMAs)
            mbar_init(smem_u32(&bars->full[s]), DIRECT ? 2 : 9);
            mbar_init(smem_u32(&bars->empty[s]), 1);
            mbar_init(smem_u32(&bars->p_full[s]), 1);
            mbar_init(smem_u32(&bars->p_empty[s]), 4);
        }
        mbar_init(smem_u32(&bars->d_full), 1);
        mbar_init(smem_u32(&bars->d_empty), 8 * p.epi_groups);     // one arrival per epilogue warp of both CTAs
        mbar_init(smem_u32(&bars->drain), 1);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_train); prefetch_tmap(&tmap_val1); prefetch_tmap(&tmap_val2);
    }
    if (p.task_off != nullptr)
        for (int j = threadIdx.x; j <= p.T; j += (int)blockDim.x) bars->task_off[j] = p.task_off[j];
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&bars->tmem_base), 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    if (FP4) {
        // unit scale factors: 0x7F in every byte of 16 tensor-memory columns behind the accumulator, all 128 lanes
        if (warp >= 6 && warp < 10) {
            uint32_t v[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = 0x7F7F7F7Fu;
            tmem_st_x16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + A_TMEM_COL, v);
            tmem_wait_st();
            tc_fence_before();
        }
        __syncthreads();         // the unpack warps' first arrival (which the first MMA waits for) comes after this
        tc_fence_after();
    }

    if (warp == 0) {
        // ------------------------------- TMA producer -------------------------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t tx_total = 2u * (uint32_t)((DIRECT ? A_STAGE : 0) + bh1 + bh2);   // both CTAs (TMA bytes only)
            const int64_t my_tiles = (num_tiles > pair) ? (num_tiles - pair + num_pairs - 1) / num_pairs : 0;
            const int64_t total = my_tiles * num_vt * p.C * nkb;
            // Packed train codes run ahead of the operand stages in their own ring: the load for iteration q is
            // issued as soon as ring slot q % nP is free, not when operand stage q % nS is.
            int64_t pq = 0;                     // next packed load to issue
            Ring pring;                         // its ring slot
            int p_kb = 0, p_i = 0, p_vt = 0;    // and its K block, checkpoint, validation tile and train tile
            int64_t p_tile = pair;
            // blocking = false: issue only if the ring slot is already free (one look at the barrier, no suspension)
            auto issue_packed = [&](bool blocking) -> bool {
                const uint32_t sp = pring.slot;
                if (blocking) { if (!mbar_wait(smem_u32(&bars->p_empty[sp]), pring.parity ^ 1u, abort_flag, p.timeout_word, TO_PRODUCER)) return false; }
                else if (!mbar_test_wait(smem_u32(&bars->p_empty[sp]), pring.parity ^ 1u)) return false;
                const uint32_t pfull = smem_u32(&bars->p_full[sp]);
                mbar_arrive_expect_tx(pfull, P_STAGE);
                tma_load_3d(smem_u32(sP + (size_t)sp * P_STAGE), &tmap_train, pfull, p_kb * PROW, (int32_t)(p_tile * 2 * TM + rank * TM), p_i);
                ++pq; pring.next((uint32_t)p.nP);
                if (++p_kb == nkb) { p_kb = 0; if (++p_i == p.C) { p_i = 0; if (++p_vt == num_vt) { p_vt = 0; p_tile += num_pairs; } } }
                return true;
            };
            Ring st_ring;

            for (int64_t tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                const int32_t row0 = (int32_t)(tile * 2 * TM + rank * TM);
                for (int vt = 0; vt < num_vt && ok; ++vt)
                    for (int i = 0; i < p.C && ok; ++i)
                        for (int kb = 0; kb < nkb; ++kb, ++it, st_ring.next((uint32_t)p.nS)) {
                            if (!DIRECT && !FP4) {
                                // the packed codes of this iteration must be on their way; those of the next few if a slot is free
                                while (pq <= (int64_t)it && ok) ok = issue_packed(true);
                                if (!ok) break;
                                while (pq < total && pq < (int64_t)it + p.nP && issue_packed(false)) {}
                            }
                            const int s = (int)st_ring.slot;
                            if (!mbar_wait_cluster(smem_u32(&bars->empty[s]), st_ring.parity ^ 1u, abort_flag, p.timeout_word, TO_PRODUCER)) { ok = false; break; }
                            const int fs = DIRECT ? (s & ~1) : s;                 // the pair's barrier
                            const uint32_t full = map_to_cta(smem_u32(&bars->full[fs]), 0);
                            if (rank == 0) mbar_arrive_expect_tx(smem_u32(&bars->full[fs]), tx_total);
                            uint8_t* st = sS + (size_t)s * stage_bytes;
                            if (DIRECT) tma_load_3d_pair(smem_u32(st), &tmap_train, full, kb * KB, row0, i);
                            // this CTA's rows of the validation operand of each MMA half
                            tma_load_3d_pair(smem_u32(st + A_SMEM), &tmap_val1, full, kb * KB, vt * p.vpad + (int)rank * (p.n1 / 2), i);
                            if (p.n2 > 0)
                                tma_load_3d_pair(smem_u32(st + A_SMEM + bh1), &tmap_val2, full, kb * KB, vt * p.vpad + p.n1 + (int)rank * (p.n2 / 2), i);
                        }
            }
            // an odd number of stages in all: the last pair's barrier still lacks its second arrival
            if (DIRECT && ok && (it & 1u) && rank == 0) mbar_arrive(smem_u32(&bars->full[st_ring.slot & ~1u]));
            if (!ok) {
                // Leave no copy in flight behind us. Packed loads 0 .. pq-1 have been issued into this CTA's own ring
                // (barriers of its own: wait, bounded, for the phases of the last nP of them). Operand stages 0 .. it-1
                // have been armed; their copies complete on the leader's barriers, whose phases also need the unpack
                // warps' arrivals at the sub-byte widths and may therefore never close: the leader gives them a bounded
                // wait, the peer idles, and neither leaves before the other (the cluster barrier at the end).
                if (!DIRECT && !FP4)
                    for (int64_t j = (pq > p.nP ? pq - p.nP : 0); j < pq; ++j)
                        if (!mbar_wait_quiet(smem_u32(&bars->p_full[j % p.nP]), (uint32_t)(j / p.nP) & 1u)) break;
                if (rank == 0) {
                    for (uint32_t j = (it > (uint32_t)p.nS ? it - (uint32_t)p.nS : 0u); j < it; ++j)
                        if (!mbar_wait_quiet(smem_u32(&bars->full[(j % (uint32_t)p.nS) & (DIRECT ? ~1u : ~0u)]), (j / (uint32_t)p.nS) & 1u, 1u << 14)) break;
                } else {
                    for (uint32_t t = 0; t < (1u << 14); ++t) __nanosleep(64);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------- MMA issuer (leader CTA) -------------------------------
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, n_acc = 0;
            Ring st_ring;
            bool ok = true;
            for (int64_t tile = pair; tile < num_tiles && ok; tile += num_pairs)
                for (int vt = 0; vt < num_vt && ok; ++vt)
                    for (int i = 0; i < p.C && ok; ++i, ++n_acc) {
                        if (!mbar_wait_cluster(smem_u32(&bars->d_empty), (n_acc & 1u) ^ 1u, abort_flag, p.timeout_word, TO_MMA)) { ok = false; break; }
                        for (int kb = 0; kb < nkb; ++kb, ++it, st_ring.next((uint32_t)p.nS)) {
                            const int s = (int)st_ring.slot;
                            if (!DIRECT || (s & 1) == 0) {       // DIRECT: the barrier at the even slot covers this stage and the next
                                // e2m1 path: the peer's unpack warps wrote their rows of A into the peer's shared memory and
                                // released them at cluster scope; tensor-memory operands are ordered by the tcgen05 fences
                                const bool okw = FP4 ? mbar_wait_cluster(smem_u32(&bars->full[s]), st_ring.parity, abort_flag, p.timeout_word, TO_MMA)
                                                     : mbar_wait(smem_u32(&bars->full[s]), st_ring.parity, abort_flag, p.timeout_word, TO_MMA);
                                if (!okw) { ok = false; break; }
                                tc_fence_after();
                            }
                            const uint32_t st = smem_u32(sS + (size_t)s * stage_bytes);
                            const uint64_t adesc = make_smem_desc_sw128(st);
                            const uint64_t bdesc1 = make_smem_desc_sw128(st + A_SMEM);
                            const uint64_t bdesc2 = make_smem_desc_sw128(st + A_SMEM + bh1);
                            const uint32_t a_tmem = tmem_base + A_TMEM_COL + (it & 1u) * 32;
#pragma unroll
                            for (int k = 0; k < KB / 32; ++k) {
                                const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                                if (BITS == 16) {
                                    mma_f16_ss_pair(tmem_base, adesc + (uint64_t)(k * 2), bdesc1 + (uint64_t)(k * 2), idesc1, acc);
                                    if (p.n2 > 0) mma_f16_ss_pair(tmem_base + p.n1, adesc + (uint64_t)(k * 2), bdesc2 + (uint64_t)(k * 2), idesc2, acc);
                                } else if (BITS == 8) {
                                    mma_i8_ss_pair(tmem_base, adesc + (uint64_t)(k * 2), bdesc1 + (uint64_t)(k * 2), idesc1, acc);
                                    if (p.n2 > 0) mma_i8_ss_pair(tmem_base + p.n1, adesc + (uint64_t)(k * 2), bdesc2 + (uint64_t)(k * 2), idesc2, acc);
                                } else if (FP4) {
                                    mma_mxf4_ss_pair(tmem_base, adesc + (uint64_t)(k * 2), bdesc1 + (uint64_t)(k * 2), idesc1, tmem_base + A_TMEM_COL, acc);
                                    if (p.n2 > 0) mma_mxf4_ss_pair(tmem_base + p.n1, adesc + (uint64_t)(k * 2), bdesc2 + (uint64_t)(k * 2), idesc2, tmem_base + A_TMEM_COL, acc);
                                } else {
                                    mma_i8_ts_pair(tmem_base, a_tmem + k * 8, bdesc1 + (uint64_t)(k * 2), idesc1, acc);
                                    if (p.n2 > 0) mma_i8_ts_pair(tmem_base + p.n1, a_tmem + k * 8, bdesc2 + (uint64_t)(k * 2), idesc2, acc);
                                }
                            }
                            mma_commit_pair(smem_u32(&bars->empty[s]));
                        }
                        if (ok) mma_commit_pair(smem_u32(&bars->d_full));
                    }
            // Whatever ended the loops, every MMA issued above completes before tensor memory is freed: one more commit
            // on a barrier of its own and a bounded wait for it (after a failed wait this covers MMAs that no commit had
            // followed; otherwise it is the wait for the last accumulator, which the epilogue needs anyway).
            mma_commit_pair(smem_u32(&bars->drain));
            mbar_wait_quiet(smem_u32(&bars->drain), 0u);
        }
    } else if (!DIRECT && (warp < 6 || (warp >= 10 && (!FP4 || warp < 10 + 4 * (fp4_groups(BITS) - 1))))) {
        // ------------------------------- unpack warps (4- and 2-bit train codes) -------------------------------
        // two groups of four warps (2-5 and 10-13) take alternate K blocks, so that the barrier round trips of
        // one block overlap the unpacking of the next
        if (FP4) {
            // 2- and 1-bit codes. A thread owns a row of the half tile and takes its packed codes straight from global memory
            // (32 or 64 bytes per K block: whole sectors), two of its group's K blocks ahead in registers; it expands them to
            // e2m1 and writes the row into operand stage s of this CTA's shared memory as the MMA reads a K-major operand
            // with the 128-byte swizzle (what a TMA load would have written): 16-byte piece j of row r at piece j ^ (r & 7).
            const int row = ((warp - 2) & 3) * 32 + lane;
            constexpr int NG = fp4_groups(BITS);                  // groups of four warps: 2-5, 10-13, 14-17, ...; group g takes K blocks g, g + NG, ...
            const uint32_t grp = (warp >= 10) ? (uint32_t)((warp - 6) >> 2) : 0u;
            constexpr int NV = PROW >= 16 ? PROW / 16 : 1;       // (this branch is compiled for every width)
            const int64_t my_tiles = (num_tiles > pair) ? (num_tiles - pair + num_pairs - 1) / num_pairs : 0;
            const int64_t total = my_tiles * num_vt * p.C * nkb;
            const int64_t row_bytes = (int64_t)p.d * BITS / 8;
            struct Pos { int kb, i, vt; int64_t tile; };
            auto advance = [&](Pos& q, int n) {
                q.kb += n;
                while (q.kb >= nkb) { q.kb -= nkb; if (++q.i == p.C) { q.i = 0; if (++q.vt == num_vt) { q.vt = 0; q.tile += num_pairs; } } }
            };
            auto fetch = [&](const Pos& q, uint4 (&r)[NV]) {
                const int64_t t = q.tile * 2 * TM + rank * TM + row;
                const uint8_t* src = p.train_codes + (int64_t)q.i * p.train_stride + t * row_bytes + (int64_t)q.kb * PROW;
#pragma unroll
                for (int c = 0; c < NV; ++c)
                    r[c] = (t < p.N && (int64_t)q.kb * PROW + 16 * c < row_bytes) ? __ldcs(reinterpret_cast<const uint4*>(src) + c)
                                                                                  : make_uint4(0u, 0u, 0u, 0u);
            };
            Pos pf{0, 0, 0, pair};
            advance(pf, (int)grp);
            Ring st_ring;
            for (uint32_t j = 0; j < grp; ++j) st_ring.next((uint32_t)p.nS);
            uint4 ra[NV], rb[NV];
            int64_t g = grp;                                      // K block (in this pair's sequence) of the registers ra
            if (g < total) { fetch(pf, ra); advance(pf, NG); }
            if (g + NG < total) { fetch(pf, rb); advance(pf, NG); }
            bool ok = true;
            auto emit = [&](const uint4 (&r)[NV]) -> bool {
                uint32_t out[32];
#pragma unroll
                for (int c = 0; c < NV; ++c) {
                    const uint32_t ww[4] = {r[c].x, r[c].y, r[c].z, r[c].w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (BITS == 1) {                 // 32 sign bits -> four words of eight e2m1 codes, in order
                            fp4_from_signs16(ww[u] & 0xFFFFu, out[(c * 4 + u) * 4], out[(c * 4 + u) * 4 + 1]);
                            fp4_from_signs16(ww[u] >> 16, out[(c * 4 + u) * 4 + 2], out[(c * 4 + u) * 4 + 3]);
                        } else {                         // 16 two-bit codes -> two words of eight e2m1 codes, in order
                            fp4_from_codes2(ww[u], out[(c * 4 + u) * 2], out[(c * 4 + u) * 2 + 1]);
                        }
                    }
                }
                const int s = (int)st_ring.slot;
                // the stage is free once the MMAs of its previous use have completed (the commit arrives in both CTAs)
                bool w = mbar_wait_parked(smem_u32(&bars->empty[s]), st_ring.parity ^ 1u, abort_flag, p.timeout_word, TO_UNPACK);
                w = __all_sync(0xFFFFFFFFu, w);
                if (!w) return false;
                uint4* dst = reinterpret_cast<uint4*>(sS + (size_t)s * stage_bytes + (size_t)row * KB);
#pragma unroll
                for (int j = 0; j < 8; ++j) dst[j ^ (row & 7)] = make_uint4(out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
                fence_proxy_async_smem();      // generic-proxy writes, read by the tensor core through the async proxy
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(smem_u32(&bars->full[s]));
                    else mbar_arrive_cluster(map_to_cta(smem_u32(&bars->full[s]), 0));      // release at cluster scope
                }
#pragma unroll
                for (int j = 0; j < NG; ++j) st_ring.next((uint32_t)p.nS);
                return true;
            };
            for (; g < total && ok; g += 2 * NG) {
                ok = emit(ra);
                if (!ok) break;
                if (g + 2 * NG < total) { fetch(pf, ra); advance(pf, NG); }
                if (g + NG < total) {
                    ok = emit(rb);
                    if (!ok) break;
                    if (g + 3 * NG < total) { fetch(pf, rb); advance(pf, NG); }
                }
            }
        } else if (!DIRECT) {
            const int row = (warp & 3) * 32 + lane;               // row of this CTA's 128-row half tile = TMEM lane
            const uint32_t grp = (warp >= 10) ? 1u : 0u;
            uint32_t it = 0;
            bool ok = true;
            const int64_t my_tiles = (num_tiles > pair) ? (num_tiles - pair + num_pairs - 1) / num_pairs : 0;
            const int64_t total = my_tiles * num_vt * p.C * nkb;
            Ring st_ring, lag_ring, pring;              // operand stage of K block it, of K block it - 2, packed slot
            for (int64_t q = 0; q < total && ok; ++q, ++it, st_ring.next((uint32_t)p.nS), pring.next((uint32_t)p.nP)) {
                if (it >= 3) lag_ring.next((uint32_t)p.nS);      // lag_ring = position of K block it - 2
                if ((it & 1u) != grp) continue;
                const int sp = (int)pring.slot, s = (int)st_ring.slot;
                ok = mbar_wait(smem_u32(&bars->p_full[sp]), pring.parity, abort_flag, p.timeout_word, TO_UNPACK);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                // unpack into registers first: this needs only the packed bytes, not the TMEM slot
                const uint4* src = reinterpret_cast<const uint4*>(sP + (size_t)sp * P_STAGE + (size_t)row * PROW);
                uint32_t out[32];
#pragma unroll
                for (int c = 0; c < PROW / 16; ++c) {
                    const uint4 w = src[c];
                    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (BITS == 4) {
                            unpack4(ww[u], out[(c * 4 + u) * 2], out[(c * 4 + u) * 2 + 1]);
                        }
                    }
                }
                // the slot is refilled by TMA (async proxy) once every reader has arrived: the reads above (generic
                // proxy, their values not yet consumed) have to be ordered before that write
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars->p_empty[sp]));      // staging slot read: the producer may refill it
                // TMEM slot it % 2 is free once the MMAs of K block it - 2 have completed, which is what releases
                // operand stage (it - 2) % nS (nS > 2, so that barrier cannot run a whole phase ahead of us)
                if (it >= 2)
                    ok = mbar_wait(smem_u32(&bars->empty[lag_ring.slot]), lag_ring.parity, abort_flag, p.timeout_word, TO_UNPACK);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                // this thread's row of the A operand: TMEM lane = row, column c = codes 4c .. 4c+3 of the block
                const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + A_TMEM_COL + (it & 1u) * 32;
                {
                    uint32_t lo16[16], hi16[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) { lo16[c] = out[c]; hi16[c] = out[16 + c]; }
                    tmem_st_x16(taddr, lo16);
                    tmem_st_x16(taddr + 16, hi16);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_leader_tmem(smem_u32(&bars->full[s]), rank);
            }
        }
    } else if ((warp >= 6 && warp < 10) || ((FP4 ? warp >= 10 : warp < 6) && p.epi_groups == 2)) {
        // ------------------------------- epilogue -------------------------------
        // warps 6-9 (group 0) and, for 8-bit codes where they have nothing to unpack, warps 2-5 (group 1): with two
        // groups each reads half of the accumulator's columns, which halves the time the tensor pipe waits for it
        const int q = warp & 3;
        const int tl = q * 32 + lane;                        // row of the tile = TMEM lane
        const int eg = (warp >= 6 && warp < 10) ? 0 : 1;
        const int et = eg * 128 + tl;                        // index among the epilogue threads
        const int nthr_e = 128 * p.epi_groups;
        const int nch = (p.vpad + 31) / 32;                  // 32-column chunks of the accumulator
        const int ch_lo = (p.epi_groups == 2 && eg == 1) ? (nch + 1) / 2 : 0;
        const int ch_hi = (p.epi_groups == 2 && eg == 0) ? (nch + 1) / 2 : nch;
        uint32_t n_acc = 0;
        bool ok = true;
        for (int64_t tile = pair; tile < num_tiles && ok; tile += num_pairs) {
            const int64_t t = tile * 2 * TM + rank * TM + tl;
            float A[TMAX];
#pragma unroll
            for (int j = 0; j < TMAX; ++j) A[j] = 0.0f;
            for (int vt = 0; vt < num_vt && ok; ++vt) {
                const int v0 = vt * p.vpad;
                const int vcount = min(p.vpad, p.V - v0);
                for (int i = 0; i < p.C && ok; ++i, ++n_acc) {
                    if (p.dots == nullptr) {
                        // this checkpoint's validation multipliers -> shared memory (epilogue threads only)
                        asm volatile("bar.sync 1, %0;" ::"r"(nthr_e) : "memory");
                        for (int v = et; v < p.vpad; v += nthr_e) bars->mv[v] = (v < vcount) ? p.val_mult[(int64_t)i * p.V + v0 + v] : 0.0f;
                        if (et < p.T) bars->eta_s[et] = p.eta_over_cnt[i * p.T + et];
                        asm volatile("bar.sync 1, %0;" ::"r"(nthr_e) : "memory");
                    }
                    // this row's multiplier: requested before the wait for the accumulator, so that its latency is not added
                    // to the time the tensor pipe waits for the accumulator to be read (the task weights are in shared memory)
                    const float mt = (p.dots == nullptr && t < p.N) ? p.train_mult[(int64_t)i * p.N + t] : 0.0f;
                    ok = mbar_wait_cluster(smem_u32(&bars->d_full), n_acc & 1u, abort_flag, p.timeout_word, TO_EPILOGUE);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
                    int j = 0;
                    if (p.dots == nullptr) while (j < p.T - 1 && bars->task_off[j + 1] <= v0 + ch_lo * 32) ++j;
                    int next_b = (p.dots == nullptr) ? bars->task_off[j + 1] - v0 : 0x7FFFFFFF;   // first column of task j+1
                    float task_sum = 0.0f;
#pragma unroll 1
                    for (int c0 = ch_lo * 32; c0 < ch_hi * 32; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld_x32(taddr + c0, v);
                        tmem_wait_ld();
                        if (c0 + 32 >= ch_hi * 32) {          // this warp's share of the accumulator is read: release it
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_leader_tmem(smem_u32(&bars->d_empty), rank);
                        }
                        if (p.dots != nullptr) {
                            if (t < p.N) {
#pragma unroll
                                for (int k = 0; k < 32; ++k)
                                    if (c0 + k < vcount) p.dots[t * p.V + v0 + c0 + k] = FP4 ? (int32_t)__uint_as_float(v[k]) : (int32_t)v[k];
                            }
                        } else {
                            // columns >= vcount carry a zero multiplier, so they add nothing
                            float x[32];
#pragma unroll
                            for (int k4 = 0; k4 < 8; ++k4) {
                                const float4 m4 = *reinterpret_cast<const float4*>(&bars->mv[c0 + 4 * k4]);
                                // the accumulator holds int32 dots; fp32 inner products for the 16-bit baseline; fp32 values that
                                // are exact integers (at most 4 d in magnitude) for the e2m1 path
                                auto acc_f = [](uint32_t raw) { return (BITS == 16 || BITS <= 2) ? __uint_as_float(raw) : (float)(int32_t)raw; };
                                x[4 * k4 + 0] = __fmul_rn(acc_f(v[4 * k4 + 0]), m4.x);
                                x[4 * k4 + 1] = __fmul_rn(acc_f(v[4 * k4 + 1]), m4.y);
                                x[4 * k4 + 2] = __fmul_rn(acc_f(v[4 * k4 + 2]), m4.z);
                                x[4 * k4 + 3] = __fmul_rn(acc_f(v[4 * k4 + 3]), m4.w);
                            }
                            // Sums in column order. A task that ends inside this chunk (or exactly at its start) closes
                            // with the columns before its end; the passes are straight-line code with predicated adds (a
                            // branch per column made such a chunk five times as slow as the others).
                            int k_lo = 0;
                            while (next_b < c0 + 32 && j < p.T) {
                                const int k_hi = next_b - c0;          // 0 .. 31
#pragma unroll
                                for (int k = 0; k < 32; ++k) if (k >= k_lo && k < k_hi) task_sum += x[k];
#pragma unroll
                                {
                                    const float add = task_sum * mt * bars->eta_s[j];
#pragma unroll
                                    for (int jj = 0; jj < TMAX; ++jj) if (jj == j) A[jj] += add;
                                }
                                task_sum = 0.0f;
                                ++j;
                                next_b = (j < p.T) ? bars->task_off[j + 1] - v0 : 0x7FFFFFFF;
                                k_lo = k_hi;
                            }
                            if (k_lo == 0) {
#pragma unroll
                                for (int k = 0; k < 32; ++k) task_sum += x[k];
                            } else {
#pragma unroll
                                for (int k = 0; k < 32; ++k) if (k >= k_lo) task_sum += x[k];
                            }
                        }
                    }
                    if (p.dots == nullptr && j < p.T) {
                        const float add = task_sum * mt * bars->eta_s[j];
#pragma unroll
                        for (int jj = 0; jj < TMAX; ++jj) if (jj == j) A[jj] += add;
                    }
                }
            }
            if (ok && p.dots == nullptr && p.epi_groups == 2) {      // add the second group's partial sums to the first's
                if (eg == 1) {
#pragma unroll
                    for (int jj = 0; jj < 6; ++jj) bars->comb[tl][jj] = A[jj];
                }
                asm volatile("bar.sync 3, 256;" ::: "memory");
                if (eg == 0) {
#pragma unroll
                    for (int jj = 0; jj < 6; ++jj) A[jj] += bars->comb[tl][jj];
                }
            }
            if (ok && p.dots == nullptr && t < p.N && eg == 0) {
                float best = A[0];
#pragma unroll
                for (int jj = 1; jj < TMAX; ++jj) if (jj < p.T) best = fmaxf(best, A[jj]);
                p.scores[t] = best;
                if (p.per_task) {
#pragma unroll
                    for (int jj = 0; jj < TMAX; ++jj) if (jj < p.T) p.per_task[t * p.T + jj] = A[jj];
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // neither CTA frees tensor memory or exits while its peer may still touch it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// Validation codes -> int8 [C][V][d] in the permutation the train-side unpack warps use.
template <int BITS>
__global__ void unpack_val_kernel(const uint8_t* __restrict__ codes, int64_t ckpt_stride, int32_t V, int32_t C, int32_t d,
                                  uint8_t* __restrict__ out)
{
    const int words_per_row = d * BITS / 32;
    const int64_t total = (int64_t)C * V * words_per_row;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t rowid = idx / words_per_row;
        const int wq = (int)(idx - rowid * words_per_row);
        const int64_t i = rowid / V, v = rowid - i * V;
        const uint32_t w = *reinterpret_cast<const uint32_t*>(codes + i * ckpt_stride + v * (int64_t)(d * BITS / 8) + 4 * wq);
        if (BITS == 4) {
            uint32_t* o = reinterpret_cast<uint32_t*>(out + rowid * d) + wq * 2;
            unpack4(w, o[0], o[1]);
        } else if (BITS == 1) {      // e2m1, two codes per byte: d / 2 bytes per row
            uint32_t* o = reinterpret_cast<uint32_t*>(out + rowid * (d / 2)) + wq * 4;
            fp4_from_signs16(w & 0xFFFFu, o[0], o[1]);
            fp4_from_signs16(w >> 16, o[2], o[3]);
        } else {
            uint32_t* o = reinterpret_cast<uint32_t*>(out + rowid * (d / 2)) + wq * 2;
            fp4_from_codes2(w, o[0], o[1]);
        }
    }
}

}  // namespace

bool score_tc_supported(int32_t T) { return T <= TMAX; }

size_t score_tc_workspace_bytes(int32_t V, int32_t C, int32_t d, int32_t bits)
{
    return bits >= 8 ? 0 : align_up((size_t)C * V * d, 256);
}

// a.dots != NULL: raw dots of one checkpoint. val_unpacked: workspace of score_tc_workspace_bytes (bits < 8).
qless_status launch_score_tc(const ScoreArgs& a, uint8_t* val_unpacked, unsigned int* timeout_word, cudaStream_t st)
{
    if (a.N == 0) return QLESS_OK;
    ScoreTcParams p;
    p.N = a.N; p.V = a.V; p.C = a.C; p.T = a.T; p.d = a.d; p.bits = a.bits;
    const int vpad_all = (a.V + 15) / 16 * 16;
    const int vcap = a.bits >= 8 ? 512 : A_TMEM_COL;        // sub-byte widths keep 64 TMEM columns for the A operand
    p.vpad = vpad_all < vcap ? vpad_all : vcap;
    p.n1 = p.vpad < 256 ? p.vpad : 256;
    p.n2 = p.vpad - p.n1;
    const int64_t row_bytes = (int64_t)a.d * a.bits / 8;

    // shared-memory plan: as many operand stages as fit (each: 16 KiB of train rows + this CTA's validation rows)
    const size_t budget = 227 * 1024 - 1024 - sizeof(ScoreBars) - 64;
    const bool fp4 = a.bits <= 2;                          // 2- and 1-bit codes: e2m1 operands, both from shared memory
    const size_t stage = ((a.bits >= 8 || fp4) ? (size_t)A_STAGE : 0) + (size_t)(p.vpad / 2) * KB;
    const size_t p_stage = (a.bits >= 8 || fp4) ? 0 : (size_t)TM * 16 * a.bits;      // packed staging ring: 4-bit codes only
    int nP = (a.bits >= 8 || fp4) ? 0 : 4;
    int nS = (int)((budget - (size_t)nP * p_stage) / stage);
    if (nS > MAX_STAGES) nS = MAX_STAGES;
    if (a.bits >= 8) nS &= ~1;                              // stages are handed to the MMAs in pairs
    QLESS_REQUIRE(nS >= 3, QLESS_ERR_UNSUPPORTED, "internal: not enough shared memory for two pipeline stages");
    p.nS = nS; p.nP = nP > 0 ? nP : 1;
    p.epi_groups = ((a.bits >= 8 || fp4) && a.T <= 6) ? 2 : 1;      // the second group: idle unpack warps (8-bit), four more warps (2-, 1-bit)
    const size_t smem = 1024 + (size_t)nS * stage + (size_t)nP * p_stage + sizeof(ScoreBars);

    p.train_codes = a.train; p.train_stride = a.C > 1 ? a.train_stride : 0;
    p.train_mult = a.train_mult; p.val_mult = a.val_mult; p.eta_over_cnt = a.eta_over_cnt; p.task_off = a.task_off;
    p.scores = a.scores; p.per_task = a.per_task; p.dots = a.dots; p.timeout_word = timeout_word;

    const uint8_t* val_src = a.val;
    int64_t val_row = row_bytes, val_stride = a.val_stride;
    if (a.bits < 8) {
        const int64_t total_words = (int64_t)a.C * a.V * (row_bytes / 4);
        int64_t blocks = (total_words + 255) / 256;
        if (blocks > (int64_t)sm_count() * 8) blocks = (int64_t)sm_count() * 8;
        if (a.bits == 4) unpack_val_kernel<4><<<(unsigned)blocks, 256, 0, st>>>(a.val, a.val_stride, a.V, a.C, a.d, val_unpacked);
        else if (a.bits == 1) unpack_val_kernel<1><<<(unsigned)blocks, 256, 0, st>>>(a.val, a.val_stride, a.V, a.C, a.d, val_unpacked);
        else unpack_val_kernel<2><<<(unsigned)blocks, 256, 0, st>>>(a.val, a.val_stride, a.V, a.C, a.d, val_unpacked);
        count_launches(1);
        val_row = fp4 ? a.d / 2 : a.d;
        val_src = val_unpacked; val_stride = (int64_t)a.V * val_row;
    }
    CUtensorMap tm_train, tm_v1, tm_v2;
    qless_status s;
    const int64_t tstride = a.C > 1 ? a.train_stride : (int64_t)a.N * row_bytes;
    s = make_tmap_3d_u8(&tm_train, a.train, (uint64_t)row_bytes, (uint64_t)a.N, (uint64_t)a.C, (uint64_t)row_bytes,
                        (uint64_t)tstride, a.bits >= 8 ? 128 : (fp4 ? 32 : 16) * a.bits, TM, a.bits >= 8);     // this CTA's 128 rows
    if (s != QLESS_OK) return s;
    const int64_t vstride = a.C > 1 ? val_stride : (int64_t)a.V * val_row;
    s = make_tmap_3d_u8(&tm_v1, val_src, (uint64_t)val_row, (uint64_t)a.V, (uint64_t)a.C, (uint64_t)val_row, (uint64_t)vstride, 128, p.n1 / 2, true);
    if (s != QLESS_OK) return s;
    s = make_tmap_3d_u8(&tm_v2, val_src, (uint64_t)val_row, (uint64_t)a.V, (uint64_t)a.C, (uint64_t)val_row, (uint64_t)vstride, 128,
                        p.n2 > 0 ? p.n2 / 2 : 8, true);
    if (s != QLESS_OK) return s;

    const int64_t tiles = (a.N + 2 * TM - 1) / (2 * TM);
    int64_t grid = (sm_count() / 2) * 2;            // CTA pairs
    if (grid > 2 * tiles) grid = 2 * tiles;
#define QLESS_LAUNCH_SCORE_TC(B)                                                                                    \
    QLESS_CUDA_TRY(cudaFuncSetAttribute(score_tc_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
    score_tc_kernel<B><<<(unsigned)grid, (B <= 2 ? fp4_threads(B) : NTHREADS), smem, st>>>(tm_train, tm_v1, tm_v2, p);
    if (a.bits == 16) { QLESS_LAUNCH_SCORE_TC(16) }
    else if (a.bits == 8) { QLESS_LAUNCH_SCORE_TC(8) }
    else if (a.bits == 4) { QLESS_LAUNCH_SCORE_TC(4) }
    else if (a.bits == 1) { QLESS_LAUNCH_SCORE_TC(1) }
    else { QLESS_LAUNCH_SCORE_TC(2) }
#undef QLESS_LAUNCH_SCORE_TC
    count_launches(1);
    QLESS_CUDA_TRY(cudaGetLastError());
    return QLESS_OK;
}

}  // namespace qless
