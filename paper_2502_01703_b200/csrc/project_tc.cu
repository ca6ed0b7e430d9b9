// Projection (Eq. 1) on the 5th-generation tensor cores.
//
//   part[s][i][r] = sum_{j in K-chunk s} Gamma[i][j] * sign(r, j)          (bf16 x bf16 -> fp32)
//
// as a GEMM with the roles chosen for the hardware. Two CTAs on neighbouring SMs form a pair and run
// one 256 x 256 x K tensor-core tile (tcgen05.mma cta_group::2). The M side (2 x 128 TMEM lanes) is a
// tile of 256 projected coordinates r, 128 per CTA, whose +-1.0 operand rows each CTA generates from
// Philox straight into its own tensor memory (no shared-memory traffic, no swizzle). The N side is a tile
// of up to 256 gradient rows, of which each CTA streams half (128 rows) by TMA from a K-blocked copy of
// Gamma ([P/64][n][64], so that each 128 x 64 operand tile is one contiguous 16 KiB span) into
// 128-byte-swizzled shared memory: pairing halves the bytes every SM pulls from L2 and the shared-memory
// traffic of the gradient operand. In each CTA the accumulator (128 x 256 fp32) occupies TMEM columns
// 0..255 and two 256-deep stages of the sign operand occupy columns 256..511 (one barrier round of the MMA-issuing
// thread covers 256 columns of both operands: 16 MMAs per two waits and two commits). Pairs are persistent and
// walk work items (gradient tile, K-chunk, r tile) K-chunk-major, so that at any time all pairs read the
// same slab of Gamma (L2 reuse); after each K-chunk the accumulator is drained to a per-chunk partial,
// which bounds the length of any fp32 accumulation chain and makes the final sum order fixed.
//
// Warp roles (448 threads per CTA; 704 for the Gaussian matrix, whose generator has eight more warps, 14-21): warp 0
// TMA producer, warp 1 MMA issuer (leader CTA only; + TMEM allocation in both), warps 2-5 and 10-13 sign generators,
// warps 6-9 accumulator drain. The leader's barriers
// collect the arrivals of both CTAs; tcgen05.commit releases stages in both CTAs at once. All waits are
// bounded; a wait that gives up raises the device timeout word and every role leaves its loop.
#include "qless_kernels.h"
#include "tc_common.cuh"

namespace qless {

namespace {

using namespace tc;

constexpr int BM = 128;                 // projected coordinates per CTA (UMMA M = 256 per pair)
constexpr int BN = 256;                 // gradient rows per tile (UMMA N), 128 of them staged by each CTA
constexpr int BK = 256;                 // K per shared-memory stage: four 64-column (128-byte) swizzle panels
constexpr int SB = 3;                   // shared-memory stages of the gradient operand
constexpr int SA = 2;                   // TMEM stages of the sign operand, 256 K each (128 columns): one per generator group
constexpr int B_PANEL_BYTES = (BN / 2) * 64 * 2;      // 16 KiB: 128 rows x 64 columns
constexpr int B_STAGE_BYTES = (BK / 64) * B_PANEL_BYTES;      // 64 KiB per CTA
constexpr int TMEM_COLS = 512;
constexpr int D_COL = 0, A_COL = 256;
constexpr int NTHREADS = 448;
constexpr int NTHREADS_GAUSS = 704;     // the Gaussian matrix: eight more generator warps (14-21)
constexpr uint32_t IDESC = make_idesc(/*D=F32*/ 1, /*A=BF16*/ 1, /*B=BF16*/ 1, 2 * BM, BN);

struct __align__(8) Barriers {
    uint64_t b_full[SB], b_empty[SB], a_full[SA], a_empty[SA], d_full, d_empty, drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
};

constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)SB * B_STAGE_BYTES + sizeof(Barriers);

// GAUSS = false: the Rademacher matrix of the method; true: Gaussian entries (Box-Muller on Philox words, bf16),
// which cost the generator warps about twenty instructions per entry instead of one.
template <bool GAUSS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GAUSS ? NTHREADS_GAUSS : NTHREADS, 1)
project_tc_kernel(const __grid_constant__ CUtensorMap tmap_gamma, int64_t n, int32_t d, int64_t P, int64_t chunk,
                  int32_t num_chunks, uint32_t kblk_base, uint64_t seed, float* __restrict__ part,
                  unsigned int* __restrict__ timeout_word)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);    // 1 KiB aligned, still a shared pointer
    Barriers* bars = reinterpret_cast<Barriers*>(smem + (size_t)SB * B_STAGE_BYTES);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = leader of the pair
    const int64_t pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_dt = (d + 2 * BM - 1) / (2 * BM);     // tiles of 256 projected coordinates
    const int num_nt = (int)((n + BN - 1) / BN);
    const int64_t num_items = (int64_t)num_nt * num_chunks * num_dt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < SB; ++s) { mbar_init(smem_u32(&bars->b_full[s]), 1); mbar_init(smem_u32(&bars->b_empty[s]), 1); }
        // a_full / d_empty of the leader collect one arrival per generator / drain warp of both CTAs
        for (int s = 0; s < SA; ++s) { mbar_init(smem_u32(&bars->a_full[s]), GAUSS ? 16 : 8); mbar_init(smem_u32(&bars->a_empty[s]), 1); }
        mbar_init(smem_u32(&bars->d_full), 1);
        mbar_init(smem_u32(&bars->d_empty), 8);
        mbar_init(smem_u32(&bars->drain), 1);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_gamma);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&bars->tmem_base), TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // both CTAs' barriers are initialised before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------- TMA producer -------------------------------
        if (lane == 0) {
            uint32_t it = 0;     // global stage counter
            bool ok = true;
            for (int64_t item = pair; item < num_items && ok; item += num_pairs) {
                const int64_t nt = item / ((int64_t)num_chunks * num_dt);
                const int kc = (int)((item / num_dt) % num_chunks);
                const int64_t k0 = (int64_t)kc * chunk;
                const int64_t klen = min(P, k0 + chunk) - k0;              // multiple of 128
                const int nkb = (int)((klen + BK - 1) / BK);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % SB;
                    const uint32_t ph = (it / SB) & 1u;
                    if (!mbar_wait_cluster(smem_u32(&bars->b_empty[s]), ph ^ 1u, abort_flag, timeout_word, TO_PRODUCER)) { ok = false; break; }
                    // both halves of the stage complete on the leader's barrier, which expects their sum
                    const int panels = (int)min((int64_t)(BK / 64), (klen - (int64_t)kb * BK) >> 6);   // a chunk may end on half a stage
                    const uint32_t full = map_to_cta(smem_u32(&bars->b_full[s]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&bars->b_full[s]), 2 * panels * B_PANEL_BYTES);
                    // tiled Gamma: K block kb64 holds its n rows of 64 columns contiguously; this CTA takes
                    // rows [rank*128, rank*128 + 128) of the 256-row tile
                    const int64_t kb64 = (k0 >> 6) + (BK / 64) * kb;
                    for (int h = 0; h < panels; ++h)
                        tma_load_2d_pair(smem_u32(smem + (size_t)s * B_STAGE_BYTES + h * B_PANEL_BYTES), &tmap_gamma, full, 0,
                                         (int32_t)((kb64 + h) * n + nt * BN + rank * (BN / 2)));
                }
            }
            if (!ok) {
                // Leave no copy in flight behind us. Stages 0 .. it-1 have been armed; all but the last SB of them were
                // consumed before their slot was armed again. Every copy of the pair completes on the leader's barrier,
                // so the leader waits (bounded) for the phases of those last stages; the peer cannot see that barrier
                // and idles instead, and leaves only after the leader does (the cluster barrier at the end).
                if (rank == 0) {
                    for (uint32_t j = (it > (uint32_t)SB ? it - SB : 0u); j < it; ++j)
                        if (!mbar_wait_quiet(smem_u32(&bars->b_full[j % SB]), (j / SB) & 1u)) break;
                } else {
                    for (uint32_t t = 0; t < (1u << 14); ++t) __nanosleep(64);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------- MMA issuer -------------------------------
        if (lane == 0 && rank == 0) {
            uint32_t itb = 0, n_item = 0;
            bool ok = true;
            for (int64_t item = pair; item < num_items && ok; item += num_pairs, ++n_item) {
                const int kc = (int)((item / num_dt) % num_chunks);
                const int64_t k0 = (int64_t)kc * chunk;
                const int64_t klen = min(P, k0 + chunk) - k0;
                const int nkb = (int)((klen + BK - 1) / BK);
                if (!mbar_wait_cluster(smem_u32(&bars->d_empty), (n_item & 1u) ^ 1u, abort_flag, timeout_word, TO_MMA)) { ok = false; break; }
                tc_fence_after();
                for (int kb = 0; kb < nkb; ++kb, ++itb) {
                    const int sb = itb % SB;
                    if (!mbar_wait(smem_u32(&bars->b_full[sb]), (itb / SB) & 1u, abort_flag, timeout_word, TO_MMA)) { ok = false; break; }
                    // the sign operand of the same 256 columns (a chunk may end on half a stage: 8 MMAs instead of 16)
                    const int nh = (int)min((int64_t)(BK / 128), (klen - (int64_t)kb * BK) >> 7);
                    const int sa = itb % SA;
                    if (!mbar_wait(smem_u32(&bars->a_full[sa]), (itb / SA) & 1u, abort_flag, timeout_word, TO_MMA)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = tmem_base + A_COL + sa * 128;
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        if (k < 8 * nh) {
                            const uint64_t bdesc = make_smem_desc_sw128(smem_u32(smem + (size_t)sb * B_STAGE_BYTES + (k >> 2) * B_PANEL_BYTES));
                            mma_f16_ts_pair(tmem_base + D_COL, a_addr + k * 8, bdesc + (uint64_t)((k & 3) * 2), IDESC, (kb > 0 || k > 0) ? 1u : 0u);
                        }
                    }
                    mma_commit_pair(smem_u32(&bars->a_empty[sa]));
                    mma_commit_pair(smem_u32(&bars->b_empty[sb]));
                }
                if (ok) mma_commit_pair(smem_u32(&bars->d_full));
            }
            // Whatever ended the loop, every MMA issued above completes before tensor memory is freed: one more commit
            // on a barrier of its own and a bounded wait for it (after the last item this is the wait for that item's
            // MMAs, which the drain warps need anyway; after a failed wait it covers MMAs that no commit had followed).
            mma_commit_pair(smem_u32(&bars->drain));
            mbar_wait_quiet(smem_u32(&bars->drain), 0u);
        }
    } else if (warp < 6 || warp >= 10) {
        // ------------------------------- sign generators -------------------------------
        // two groups of four warps (2-5 and 10-13) take alternate 256-deep stages (each group owns one of the two
        // TMEM stages), so that the latency of one stage (Philox chains, TMEM stores, barrier round trip) overlaps the next
        // (Gaussian matrix: the entries cost twenty times as many instructions, so each stage has eight warps, two per
        // quadrant: warps 2-5 and 10-13 generate the first 128 columns of their group's stage, warps 14-17 and 18-21 the second)
        const int q = warp & 3;                                  // TMEM lane quadrant this warp may access
        const uint32_t grp = (warp >= 18) ? 1u : (warp >= 14) ? 0u : (warp >= 10) ? 1u : 0u;
        const int my_half = (warp >= 14) ? 1 : 0;
        uint32_t ita = 0;
        bool ok = true;
        for (int64_t item = pair; item < num_items && ok; item += num_pairs) {
            const int dt = (int)(item % num_dt) * 2 + (int)rank;           // this CTA's 128 projected coordinates
            const int kc = (int)((item / num_dt) % num_chunks);
            const int64_t k0 = (int64_t)kc * chunk;
            const int64_t klen = min(P, k0 + chunk) - k0;                  // multiple of 128
            const int nka = (int)((klen + BK - 1) / BK);                   // 256-deep stages of the chunk
            const uint32_t r = (uint32_t)(dt * BM + q * 32 + lane);
            for (int ka = 0; ka < nka; ++ka, ++ita) {
                if ((ita & 1u) != grp) continue;
                const int sa = ita % SA;                                   // = grp: each group owns one stage
                const int nh = (int)min((int64_t)2, (klen - (int64_t)ka * BK) >> 7);      // halves of 128 columns (a chunk may end on one)
                const uint32_t blk = kblk_base + (uint32_t)((k0 >> 7) + 2 * ka);          // first 128-column block of the stage
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + A_COL + sa * 128;
                if constexpr (GAUSS) {
                    const int h = my_half;
                    uint32_t v[4][16];                                            // generated before the slot is waited for
                    if (h < nh) {
                        const uint32_t bh = blk + (uint32_t)h;
#pragma unroll
                        for (int wi = 0; wi < 4; ++wi)
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                gaussian_quad_bf16x2(seed, r, (bh << 5) | (uint32_t)(wi * 8 + c), bh >> 27, v[wi][2 * c], v[wi][2 * c + 1]);
                    }
                    // a warp with nothing to generate (the chunk ends on half a stage) still waits before it arrives: its
                    // arrival must not land in the stage's previous phase
                    ok = mbar_wait_cluster(smem_u32(&bars->a_empty[sa]), ((ita / SA) & 1u) ^ 1u, abort_flag, timeout_word, TO_GENERATOR);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    if (h < nh) {
#pragma unroll
                        for (int wi = 0; wi < 4; ++wi) tmem_st_x16(taddr + h * 64 + wi * 16, v[wi]);
                    }
                } else {
                    uint32_t w[2][4];
                    rademacher_block(seed, r, blk, w[0]);     // overlaps with the wait below
                    if (nh == 2) rademacher_block(seed, r, blk + 1u, w[1]);
                    ok = mbar_wait_cluster(smem_u32(&bars->a_empty[sa]), ((ita / SA) & 1u) ^ 1u, abort_flag, timeout_word, TO_GENERATOR);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h < nh) {
#pragma unroll
                            for (int wi = 0; wi < 4; ++wi) {
                                uint32_t v[16];
#pragma unroll
                                for (int p = 0; p < 16; ++p) v[p] = rademacher_bf16x2(w[h][wi], p);
                                tmem_st_x16(taddr + h * 64 + wi * 16, v);
                            }
                        }
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_leader_tmem(smem_u32(&bars->a_full[sa]), rank);
            }
        }
    } else {
        // ------------------------------- accumulator drain -------------------------------
        const int q = warp & 3;
        uint32_t n_item = 0;
        bool ok = true;
        for (int64_t item = pair; item < num_items && ok; item += num_pairs, ++n_item) {
            const int dt = (int)(item % num_dt) * 2 + (int)rank;
            const int kc = (int)((item / num_dt) % num_chunks);
            const int64_t nt = item / ((int64_t)num_chunks * num_dt);
            ok = mbar_wait_cluster(smem_u32(&bars->d_full), n_item & 1u, abort_flag, timeout_word, TO_EPILOGUE);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            float* out = part + ((int64_t)kc * n + nt * BN) * d + dt * BM + q * 32 + lane;
            const int64_t rows_here = (dt * BM < d) ? min((int64_t)BN, n - nt * BN) : 0;   // d = 128 (mod 256): last half tile is empty
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + D_COL;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                tmem_ld_x32(taddr + c0, v);
                tmem_wait_ld();
                if (c0 + 32 == BN) {          // accumulator fully read: hand it back before the stores
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_leader_tmem(smem_u32(&bars->d_empty), rank);
                }
#pragma unroll
                for (int k = 0; k < 32; ++k)
                    if (c0 + k < rows_here) __stcs(out + (int64_t)(c0 + k) * d, __uint_as_float(v[k]));
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // neither CTA frees tensor memory or exits while its peer may still touch it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace

size_t project_tc_smem_bytes() { return SMEM_BYTES; }

cudaError_t launch_project_tc(const CUtensorMap& tmap, const ProjectPlan& pl, uint64_t seed, float* part,
                              unsigned int* timeout_word, cudaStream_t st)
{
    if (pl.n == 0) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(pl.gaussian ? project_tc_kernel<true> : project_tc_kernel<false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int64_t items = (int64_t)((pl.n + BN - 1) / BN) * pl.num_chunks * ((pl.d + 2 * BM - 1) / (2 * BM));
    int64_t grid = (sm_count() / 2) * 2;               // CTA pairs
    if (grid > 2 * items) grid = 2 * items;
    if (pl.gaussian)
        project_tc_kernel<true><<<(unsigned)grid, NTHREADS_GAUSS, SMEM_BYTES, st>>>(tmap, pl.n, pl.d, pl.P, pl.chunk, pl.num_chunks,
                                                                              (uint32_t)(pl.k_base >> 7), seed, part, timeout_word);
    else
        project_tc_kernel<false><<<(unsigned)grid, NTHREADS, SMEM_BYTES, st>>>(tmap, pl.n, pl.d, pl.P, pl.chunk, pl.num_chunks,
                                                                               (uint32_t)(pl.k_base >> 7), seed, part, timeout_word);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace qless
