// Stage 4: top-k by radix select on order-preserving 32-bit keys, then an index-ordered compaction.
// The k-th largest key T and the number of keys equal to T that are admitted (smallest indices first) are
// found exactly; the compaction writes the indices of {key > T} and of the admitted ties in ascending order.
// Three designs by size: one cluster launch that keeps the keys in shared memory (up to 360 448 scores), a
// multi-pass radix select on the scores (up to 2^22), and above that a sampled two-sided bracket of T with one
// streaming pass over the scores.
#include <cmath>
#include <mutex>

#include "qless_kernels.h"
#include "tc_common.cuh"

namespace qless {

namespace {

constexpr int SEL_T = 256;
constexpr int SEL_EPT = 8;                       // elements per thread in the compaction
constexpr int SEL_CHUNK = SEL_T * SEL_EPT;       // 2048 elements per unit of the compaction
constexpr int SEL_MAX_GRID = 1024;               // blocks of the count and write kernels (one total per block)

struct SelectState {
    uint32_t prefix;      // key bits fixed so far (right-aligned)
    uint32_t pad;
    int64_t k_rem;        // how many more to take from the current bucket
    uint32_t ticket[4];   // blocks that have finished each histogram round (the last one scans)
};

// Workspace: histograms | state (256 B) | block totals | unit counts (2 x int32 per 2048-score unit)
struct SelectWs {
    uint32_t* hist;       // [3][2048]
    SelectState* state;
    int64_t* blk_tot;     // [SEL_MAX_GRID][2]  totals (gt, eq) of each block's range of units
    int32_t* blk_cnt;     // [nblk][2]  (gt, eq) per unit
};

// A kernel whose gate is closed returns at once: the launches of the bracketed path and of its
// fallback are both enqueued, and a flag written on the device decides which of the two does the work.
struct Gate {
    const uint32_t* flag;     // nullptr: always open
    uint32_t want;
    __device__ __forceinline__ bool closed() const { return flag != nullptr && *flag != want; }
};

__host__ __device__ inline int64_t sel_nblk(int64_t N) { return (N + SEL_CHUNK - 1) / SEL_CHUNK; }

// Programmatic dependent launch: a kernel launched with launch_after() may be set up on the GPU while the kernel before
// it in the stream is still draining; its first statement, dep_wait(), returns only when that kernel has completed and
// its writes are visible, so nothing it reads can be stale. dep_release() right after lets the launch behind start
// its own set-up in the same way. (Both are no-ops in a kernel launched the ordinary way.)
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_after(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The block (256 threads) that finishes a histogram round last finds the bin that holds the k_rem-th largest key,
// counting from the top bin down: thread t owns NB / 256 consecutive bins from the top. Returns false if the
// histogram holds fewer than k_rem keys. hist is read around L1 (other blocks' atomics filled it).
template <int NB>
__device__ __forceinline__ bool block_find_bin(const uint32_t* hist, int64_t k_rem, uint32_t* bin_out, int64_t* krem_out)
{
    constexpr int PER = NB / SEL_T;
    __shared__ int64_t s_w[SEL_T / 32];
    __shared__ uint32_t s_bin;
    __shared__ int64_t s_krem;
    __shared__ int s_found;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_found = 0;
    uint32_t c[PER];
    int64_t mine = 0;
#pragma unroll
    for (int u = 0; u < PER; ++u) { c[u] = __ldcg(hist + (NB - 1 - (tid * PER + u))); mine += c[u]; }
    int64_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t a = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += a;
    }
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    int64_t pre = inc - mine;
    for (int w = 0; w < warp; ++w) pre += s_w[w];
#pragma unroll
    for (int u = 0; u < PER; ++u) {
        if (pre < k_rem && k_rem <= pre + c[u]) {       // at most one (thread, u) satisfies this
            s_bin = (uint32_t)(NB - 1 - (tid * PER + u));
            s_krem = k_rem - pre;
            s_found = 1;
        }
        pre += c[u];
    }
    __syncthreads();
    *bin_out = s_bin; *krem_out = s_krem;
    return s_found != 0;
}

// All threads of a block call this after their last global atomic of a round: true in every thread of the block
// that arrives last (its reads then see every other block's contributions).
__device__ __forceinline__ bool last_block_done(uint32_t* ticket)
{
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    const bool last = s_last != 0;
    if (last) __threadfence();
    return last;
}

// One radix round on the scores (11 + 11 + 10 bits of the key); the last block to finish fixes the round's bits.
template <int PASS>
__device__ __forceinline__ void select_hist_body(const float* __restrict__ scores, int64_t N, int64_t k, SelectState* __restrict__ state,
                                                 uint32_t* __restrict__ hist)
{
    __shared__ uint32_t s_h[2048];
    for (int i = threadIdx.x; i < 2048; i += SEL_T) s_h[i] = 0;
    __syncthreads();
    const uint32_t prefix = (PASS == 0) ? 0u : state->prefix;
    const int64_t stride = (int64_t)gridDim.x * SEL_T;
    // vector body (4 scores per load) + scalar tail
    const int64_t n4 = N >> 2;
    for (int64_t i = (int64_t)blockIdx.x * SEL_T + threadIdx.x; i < n4; i += stride) {
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(scores) + i);
        const uint32_t kk[4] = {order_key(raw.x), order_key(raw.y), order_key(raw.z), order_key(raw.w)};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (PASS == 0) atomicAdd(&s_h[kk[u] >> 21], 1u);
            else if (PASS == 1) { if ((kk[u] >> 21) == prefix) atomicAdd(&s_h[(kk[u] >> 10) & 0x7FFu], 1u); }
            else { if ((kk[u] >> 10) == prefix) atomicAdd(&s_h[kk[u] & 0x3FFu], 1u); }
        }
    }
    for (int64_t i = (n4 << 2) + (int64_t)blockIdx.x * SEL_T + threadIdx.x; i < N; i += stride) {
        const uint32_t kk = order_key(__float_as_uint(scores[i]));
        if (PASS == 0) atomicAdd(&s_h[kk >> 21], 1u);
        else if (PASS == 1) { if ((kk >> 21) == prefix) atomicAdd(&s_h[(kk >> 10) & 0x7FFu], 1u); }
        else { if ((kk >> 10) == prefix) atomicAdd(&s_h[kk & 0x3FFu], 1u); }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2048; i += SEL_T)
        if (s_h[i]) atomicAdd(&hist[i], s_h[i]);
    if (!last_block_done(&state->ticket[PASS])) return;
    constexpr int SHIFT = (PASS == 2) ? 10 : 11;
    const int64_t k_rem = (PASS == 0) ? k : state->k_rem;
    uint32_t bin; int64_t krem;
    bool found;
    if constexpr (PASS == 2) found = block_find_bin<1024>(hist, k_rem, &bin, &krem);
    else found = block_find_bin<2048>(hist, k_rem, &bin, &krem);
    if (found && threadIdx.x == 0) { state->prefix = (prefix << SHIFT) | bin; state->k_rem = krem; }
}
template <int PASS>
__global__ void __launch_bounds__(SEL_T)
select_hist_kernel(const float* __restrict__ scores, int64_t N, int64_t k, SelectState* __restrict__ state,
                   uint32_t* __restrict__ hist)
{
    dep_wait();
    dep_release();
    select_hist_body<PASS>(scores, N, k, state, hist);
}

// Counts of {key > T} and {key == T} per 2048-score unit. Block b owns the units [b R, (b + 1) R) and leaves their
// totals, so that the write kernel needs no prefix-sum pass in between.
__device__ __forceinline__ void select_count_body(const float* __restrict__ scores, int64_t N, int64_t nblk, int64_t R, int64_t G,
                                                  const SelectState* __restrict__ state, int32_t* __restrict__ blk_cnt,
                                                  int64_t* __restrict__ blk_tot)
{
    __shared__ int s_gt[SEL_T / 32], s_eq[SEL_T / 32];
    if ((int64_t)blockIdx.x >= G) return;            // the launch may be wider than the partition
    const uint32_t T = state->prefix;
    const int64_t u0 = (int64_t)blockIdx.x * R, u1 = (u0 + R < nblk) ? u0 + R : nblk;
    int64_t tot_gt = 0, tot_eq = 0;
    for (int64_t blk = u0; blk < u1; ++blk) {
        const int64_t base = blk * SEL_CHUNK + threadIdx.x * SEL_EPT;
        int gt = 0, eq = 0;
        if (base + SEL_EPT <= N) {
            const uint4 r0 = __ldg(reinterpret_cast<const uint4*>(scores + base)), r1 = __ldg(reinterpret_cast<const uint4*>(scores + base) + 1);
            const uint32_t r[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
            for (int u = 0; u < SEL_EPT; ++u) { const uint32_t kk = order_key(r[u]); gt += (kk > T); eq += (kk == T); }
        } else {
#pragma unroll
            for (int u = 0; u < SEL_EPT; ++u) {
                const int64_t i = base + u;
                if (i < N) { const uint32_t kk = order_key(__float_as_uint(scores[i])); gt += (kk > T); eq += (kk == T); }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { gt += __shfl_xor_sync(0xFFFFFFFFu, gt, o); eq += __shfl_xor_sync(0xFFFFFFFFu, eq, o); }
        if ((threadIdx.x & 31) == 0) { s_gt[threadIdx.x >> 5] = gt; s_eq[threadIdx.x >> 5] = eq; }
        __syncthreads();
        if (threadIdx.x == 0) {
            int a = 0, b = 0;
            for (int w = 0; w < SEL_T / 32; ++w) { a += s_gt[w]; b += s_eq[w]; }
            blk_cnt[2 * blk] = a; blk_cnt[2 * blk + 1] = b;
            tot_gt += a; tot_eq += b;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) { blk_tot[2 * blockIdx.x] = tot_gt; blk_tot[2 * blockIdx.x + 1] = tot_eq; }
}
__global__ void __launch_bounds__(SEL_T)
select_count_kernel(const float* __restrict__ scores, int64_t N, int64_t nblk, int64_t R, int64_t G, const SelectState* __restrict__ state,
                    int32_t* __restrict__ blk_cnt, int64_t* __restrict__ blk_tot)
{
    dep_wait();
    dep_release();
    select_count_body(scores, N, nblk, R, G, state, blk_cnt, blk_tot);
}

// Sum of the totals of the blocks before this one (every thread gets both sums).
__device__ __forceinline__ void block_base_before(const int64_t* __restrict__ blk_tot, int64_t& base0, int64_t& base1)
{
    __shared__ int64_t s_b[2][SEL_T / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t a0 = 0, a1 = 0;
    for (int b = threadIdx.x; b < (int)blockIdx.x; b += SEL_T) { a0 += __ldcg(blk_tot + 2 * b); a1 += __ldcg(blk_tot + 2 * b + 1); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { a0 += __shfl_xor_sync(0xFFFFFFFFu, a0, o); a1 += __shfl_xor_sync(0xFFFFFFFFu, a1, o); }
    if (lane == 0) { s_b[0][warp] = a0; s_b[1][warp] = a1; }
    __syncthreads();
    base0 = 0; base1 = 0;
#pragma unroll
    for (int w = 0; w < SEL_T / 32; ++w) { base0 += s_b[0][w]; base1 += s_b[1][w]; }
    __syncthreads();
}

__global__ void __launch_bounds__(SEL_T)
select_write_kernel(const float* __restrict__ scores, int64_t N, int64_t nblk, int64_t R, const SelectState* __restrict__ state,
                    const int32_t* __restrict__ blk_cnt, const int64_t* __restrict__ blk_tot, int64_t* __restrict__ indices, Gate gate)
{
    dep_wait();
    __shared__ int s_gt[SEL_T / 32], s_eq[SEL_T / 32];
    if (gate.closed()) return;
    const uint32_t T = state->prefix;
    const int64_t k_ties = state->k_rem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t gt_run, eq_run;                   // selected-larger and tied scores before the current unit
    block_base_before(blk_tot, gt_run, eq_run);
    const int64_t u0 = (int64_t)blockIdx.x * R, u1 = (u0 + R < nblk) ? u0 + R : nblk;
    for (int64_t blk = u0; blk < u1; ++blk) {
        const int64_t base = blk * SEL_CHUNK + threadIdx.x * SEL_EPT;
        uint32_t fgt = 0, feq = 0;
#pragma unroll
        for (int u = 0; u < SEL_EPT; ++u) {
            const int64_t i = base + u;
            if (i < N) {
                const uint32_t kk = order_key(__float_as_uint(scores[i]));
                fgt |= (uint32_t)(kk > T) << u; feq |= (uint32_t)(kk == T) << u;
            }
        }
        const int gt = __popc(fgt), eq = __popc(feq);
        int igt = gt, ieq = eq;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int a = __shfl_up_sync(0xFFFFFFFFu, igt, o), b = __shfl_up_sync(0xFFFFFFFFu, ieq, o);
            if (lane >= o) { igt += a; ieq += b; }
        }
        if (lane == 31) { s_gt[warp] = igt; s_eq[warp] = ieq; }
        __syncthreads();
        int64_t gt_before = gt_run + igt - gt;
        int64_t eq_before = eq_run + ieq - eq;
        for (int w = 0; w < warp; ++w) { gt_before += s_gt[w]; eq_before += s_eq[w]; }
#pragma unroll
        for (int u = 0; u < SEL_EPT; ++u) {
            const bool g = (fgt >> u) & 1u, e = (feq >> u) & 1u;
            if (g || (e && eq_before < k_ties)) {
                const int64_t pos = gt_before + (eq_before < k_ties ? eq_before : k_ties);
                indices[pos] = base + u;
            }
            gt_before += g; eq_before += e;
        }
        gt_run += blk_cnt[2 * blk]; eq_run += blk_cnt[2 * blk + 1];
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// Large N: the scores are read once. A stratified sample (offset inside each stratum hashed) brackets the
// k-th largest key T from both sides: lo <= T <= hi except with probability below 1e-8 per side, for scores in
// any order. One streaming pass over the scores then classifies each key: above hi it is selected for sure,
// inside [lo, hi] it may be (about 2 % of N for a 5 % selection), below lo it is dropped. Per 4096-score chunk
// the pass leaves the offsets of both classes in index order (16 bits each, the class in the top bit) and, for
// the second class, (key, offset) pairs; it also counts the first class and histograms the second. T is then
// found by a radix select on the pairs alone (their keys span hi - lo, usually some 2^21 values: 8 + 12 (+ 12)
// bits), and the final write walks each chunk's ordered list, looks the second class up in a bitmap built from
// the chunk's pairs, and writes the selected indices in ascending order. If T falls outside the bracket (the
// counts show it), a flag opens the gates of the exact multi-pass path enqueued behind.
// ------------------------------------------------------------------------------------------------

constexpr int SG_T = 256;
constexpr int SG_CH = 4096;                     // scores per chunk = capacity of its lists
constexpr int SG_SAMPLE = 1 << 18;              // strata (one sampled score each): the bracket holds about 0.5 % of N at a 5 % selection
constexpr int64_t SG_MIN_N = (int64_t)1 << 22;  // above this the bracketed path is used
constexpr int B1_BINS = 256, B23_BINS = 4096;   // bins of the first round (in the streaming pass) and of the later ones

struct BracketState {
    uint32_t lo_key, hi_key;      // second class: lo <= key <= hi; first class: key > hi
    uint32_t b[3], sh[3];         // bits and right shift of the three radix rounds on rel = key - lo
    uint32_t rel_prefix;          // bits of T - lo fixed so far
    uint32_t fallback;            // 1: T lies outside the bracket, the exact path must run
    uint32_t T, pad;              // the k-th largest key, once known
    int64_t k_rem;                // rank still to find inside the current bucket; ties admitted, at the end
    unsigned long long n_sure, n_maybe;
    uint32_t s_bin[2], s_rem[2];  // sample: first-level bin of the two bracket ranks and the ranks left inside it
    uint32_t ticket[6];           // blocks that have finished: sample levels 1, 2; streaming pass; pair rounds 2, 3
};

// What the streaming pass leaves per 4096-score chunk: a bitmap of the first class (one bit per score, 512 bytes,
// consecutive chunks side by side), and the (key, offset) pairs of the second class in two levels. A chunk usually
// yields some twenty pairs but may yield 4096 (constant scores): the first PP pairs of every chunk live in dense arrays
// (the passes that read them stream through memory); whatever comes after goes to full-size segments, pair i at slot
// i, that typical inputs never touch.
constexpr int PG = 16, PU = 1;                  // pair lists a warp walks together, and loads in flight per lane and list
constexpr int PP = 32 * PU;                     // dense capacity per chunk: pairs
constexpr int BMW = SG_CH / 32;                 // bitmap words per chunk
struct ChunkLists {
    uint32_t* sure_bm;            // [nchunk][BMW]  bit (o & 31) of word o >> 5: score o of the chunk is above hi
    uint32_t* key_p;              // [nchunk][PP]   keys of the pairs (any order)
    uint32_t* key_o;              // [nchunk][SG_CH]
    uint16_t* off_p;              // [nchunk][PP]   offsets of the pairs
    uint16_t* off_o;              // [nchunk][SG_CH]
    __device__ __forceinline__ uint32_t* key(int64_t c, uint32_t i) const { return i < (uint32_t)PP ? key_p + c * PP + i : key_o + c * SG_CH + i; }
    __device__ __forceinline__ uint16_t* off(int64_t c, uint32_t i) const { return i < (uint32_t)PP ? off_p + c * PP + i : off_o + c * SG_CH + i; }
};

struct BracketWs {
    uint32_t* hist;               // [B1_BINS + 2 * B23_BINS] rounds of the bracketed path, [3][2048] of the fallback, [3][4096] of the sample
    BracketState* bstate;         // 256-byte region
    SelectState* fstate;          // 256-byte region (fallback)
    int64_t* blk_tot;             // [SEL_MAX_GRID][2]
    int32_t* blk_cnt;             // [max(chunks, fallback units)][2]
    uint32_t* sample_key;         // [SG_SAMPLE]
    uint32_t* chunk_cnt;          // [nchunk]  scores above hi | pairs << 16
    ChunkLists L;
};
constexpr int BR_HIST_WORDS = B1_BINS + 2 * B23_BINS + 3 * 2048 + 3 * 4096;

__host__ __device__ inline int64_t sg_nchunk(int64_t N) { return (N + SG_CH - 1) / SG_CH; }

__device__ __forceinline__ uint32_t mix32(uint32_t x)
{
    x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
    return x;
}

// The bracket from the sample: the sampled keys of ranks r_lo = ceil(k S / N) + w and r_hi = ceil(k S / N) - w
// (counted from the largest), w = 6 standard deviations of that rank + 8, by two radix levels of 12 bits each on the
// 262144 sampled keys, spread over 64 blocks whose last one scans. The remaining 8 bits are rounded outwards (lo
// down, hi up), which keeps both bounds valid and widens the bracket by at most 2^-15 of T's magnitude.
constexpr int SS_BLOCKS = 64, SS_PER = SG_SAMPLE / (SS_BLOCKS * SEL_T);     // blocks of the two level kernels, keys per thread
struct SampleRanks { int r_lo, r_hi; bool all_lo, no_hi; };
__device__ __forceinline__ SampleRanks sample_ranks(int64_t N, int64_t k)
{
    const double p = (double)k / (double)N;
    const double ks = ceil(p * (double)SG_SAMPLE);
    const double w = ceil(6.0 * sqrt(ks * (1.0 - p))) + 8.0;
    SampleRanks r;
    r.all_lo = ks + w >= (double)SG_SAMPLE;        // every score is a candidate
    r.no_hi = ks - w < 1.0;                        // no score is selected for sure
    r.r_lo = r.all_lo ? SG_SAMPLE : (int)(ks + w);
    r.r_hi = r.no_hi ? 1 : (int)(ks - w);
    return r;
}

// Level 1 also draws the sample: one score per stratum of N / 262144 scores, at a hashed offset inside it.
__global__ void __launch_bounds__(SEL_T)
sample_level1_kernel(const float* __restrict__ scores, uint32_t* __restrict__ sample_key, int64_t N, int64_t k,
                     BracketState* __restrict__ bs, uint32_t* __restrict__ hist)
{
    dep_wait();
    dep_release();
    __shared__ uint32_t s_h[4096];
    for (int i = threadIdx.x; i < 4096; i += SEL_T) s_h[i] = 0;
    const int64_t per = N / SG_SAMPLE;                      // >= 16 for every N this path takes
    uint32_t key[SS_PER];
#pragma unroll
    for (int i = 0; i < SS_PER; ++i) {                      // grid covers SG_SAMPLE keys; all scattered reads in flight together
        const int j = (blockIdx.x * SS_PER + i) * SEL_T + threadIdx.x;
        // offset inside the stratum: hash scaled to [0, per) (per < 2^32 for every N below 2^50)
        const int64_t pos = (int64_t)j * per + (int64_t)(((uint64_t)mix32(0x9E3779B9u * (uint32_t)j + 0x85EBCA6Bu) * (uint64_t)per) >> 32);
        key[i] = order_key(__float_as_uint(__ldg(scores + pos)));
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < SS_PER; ++i) {
        sample_key[(blockIdx.x * SS_PER + i) * SEL_T + threadIdx.x] = key[i];
        atomicAdd(&s_h[key[i] >> 20], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 4096; i += SEL_T)
        if (s_h[i]) atomicAdd(&hist[i], s_h[i]);
    if (!last_block_done(&bs->ticket[0])) return;
    const SampleRanks r = sample_ranks(N, k);
    uint32_t bin; int64_t rem;
    block_find_bin<4096>(hist, r.r_lo, &bin, &rem);
    if (threadIdx.x == 0) { bs->s_bin[0] = bin; bs->s_rem[0] = (uint32_t)rem; }
    __syncthreads();
    block_find_bin<4096>(hist, r.r_hi, &bin, &rem);
    if (threadIdx.x == 0) { bs->s_bin[1] = bin; bs->s_rem[1] = (uint32_t)rem; }
}

__global__ void __launch_bounds__(SEL_T)
sample_level2_kernel(const uint32_t* __restrict__ sample_key, int64_t N, int64_t k, BracketState* __restrict__ bs,
                     uint32_t* __restrict__ hist_lo, uint32_t* __restrict__ hist_hi, int force_short)
{
    dep_wait();
    dep_release();
    __shared__ uint32_t s_h[2][4096];
    for (int i = threadIdx.x; i < 2 * 4096; i += SEL_T) (&s_h[0][0])[i] = 0;
    __syncthreads();
    const uint32_t bin_lo = bs->s_bin[0], bin_hi = bs->s_bin[1];
    for (int i = 0; i < SS_PER; ++i) {
        const uint32_t key = sample_key[(blockIdx.x * SS_PER + i) * SEL_T + threadIdx.x];
        if ((key >> 20) == bin_lo) atomicAdd(&s_h[0][(key >> 8) & 0xFFFu], 1u);
        if ((key >> 20) == bin_hi) atomicAdd(&s_h[1][(key >> 8) & 0xFFFu], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 4096; i += SEL_T) {
        if (s_h[0][i]) atomicAdd(&hist_lo[i], s_h[0][i]);
        if (s_h[1][i]) atomicAdd(&hist_hi[i], s_h[1][i]);
    }
    if (!last_block_done(&bs->ticket[1])) return;
    const SampleRanks r = sample_ranks(N, k);
    uint32_t sub_lo, sub_hi; int64_t rem;
    block_find_bin<4096>(hist_lo, (int64_t)bs->s_rem[0], &sub_lo, &rem);
    __syncthreads();
    block_find_bin<4096>(hist_hi, (int64_t)bs->s_rem[1], &sub_hi, &rem);
    if (threadIdx.x == 0) {
        uint32_t lo = r.all_lo ? 0u : ((bin_lo << 20) | (sub_lo << 8));
        uint32_t hi = r.no_hi ? 0xFFFFFFFFu : ((bin_hi << 20) | (sub_hi << 8) | 0xFFu);
        if (force_short) lo = hi = 0xFF800000u;             // key of +inf: (almost) nothing qualifies
        if (hi < lo) hi = lo;                               // cannot happen (r_hi <= r_lo); keeps the plan below sane
        // plan of the radix rounds on key - lo, which lies in [0, hi - lo]: 8 bits in the streaming pass, then 12 and 12
        const uint32_t range = hi - lo;
        const uint32_t nbits = range ? 32u - (uint32_t)__clz((int)range) : 0u;
        const uint32_t b1 = nbits < 8u ? nbits : 8u, rest = nbits - b1, b2 = rest < 12u ? rest : 12u, b3 = rest - b2;
        bs->lo_key = lo; bs->hi_key = hi;
        bs->b[0] = b1; bs->b[1] = b2; bs->b[2] = b3;
        bs->sh[0] = nbits - b1; bs->sh[1] = nbits - b1 - b2; bs->sh[2] = 0u;
    }
}

// The one read of the scores. A warp owns whole chunks and walks each in eight steps of 512 scores, with no
// block-wide barrier. Each lane fetches four 16-byte pieces of a step with cp.async into a ring of three steps, two
// steps ahead of the one the warp works on: enough bytes in flight per SM without registers. A step is then read back
// as 16 slots of 32 consecutive scores (lane = score): two ballots per slot are the slot's words of the two class
// bitmaps, with no scan and no divergence. The first-class words go to memory as they are (64 bytes per step); the
// few set bits of the second-class words (2 % of the scores) are then turned into pairs, half a word per lane.
// The class test runs on s = key ^ 0x80000000 read as a signed integer: for a bracket above zero (MODE 0) s is the raw
// bit pattern itself, and negative scores and NaNs fall outside the range by themselves; for other brackets (MODE 1)
// s takes two more operations per score; if every score is a candidate (MODE 2, lo = 0) the key is formed in full,
// so that NaNs (key 0) land in the second class.
constexpr int SG_RING = 3;
constexpr int SG_STEP = 512;                    // scores per warp step
constexpr int SG_STEPS = SG_CH / SG_STEP;       // 8

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int KEEP> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(KEEP) : "memory"); }

template <int MODE>
__device__ __forceinline__ void gather_chunks(const float* __restrict__ scores, int64_t N, uint32_t lo, uint32_t hi, uint32_t sh1,
                                              const ChunkLists& L, uint32_t* __restrict__ chunk_cnt, uint32_t* s_h, uint32_t* s_mc /* this warp's pair counter */,
                                              uint32_t* s_w /* this warp's 32 ballot words */, uint32_t* s_ring /* this warp's [SG_RING][SG_STEP] */,
                                              unsigned long long& sure_total, unsigned long long& maybe_total)
{
    const int lane = threadIdx.x & 31;
    const uint32_t lo_s = lo ^ 0x80000000u, hi_s = hi ^ 0x80000000u;
    const uint32_t range = 0x7F800000u - lo_s;                     // up to the image of +inf (MODE 0, 1)
    const int64_t nchunk = sg_nchunk(N);
    const int64_t gwarp = (int64_t)blockIdx.x * (SG_T / 32) + (threadIdx.x >> 5);
    const int64_t nwarp = (int64_t)gridDim.x * (SG_T / 32);
    const uint32_t ring_u32 = (uint32_t)__cvta_generic_to_shared(s_ring) + lane * 16;

    // fetch cursor: two steps ahead of the work cursor
    int64_t fc = gwarp; int fsub = 0, fslot = 0;
    auto fetch = [&]() {
        if (fc < nchunk) {
            const int64_t i0 = fc * SG_CH + fsub * SG_STEP;          // first score of the step
            const float* src = scores + i0 + lane * 4;
            const uint32_t dst = ring_u32 + fslot * (SG_STEP * 4);
            if (N - i0 >= SG_STEP) {
#pragma unroll
                for (int j = 0; j < 4; ++j) cp_async16(dst + j * 512, src + j * 128, 16);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {                        // pieces beyond N are zero-filled
                    const int64_t left = N - (i0 + lane * 4 + j * 128);
                    const int nb = left >= 4 ? 16 : (left > 0 ? (int)left * 4 : 0);
                    cp_async16(dst + j * 512, nb ? (const void*)(src + j * 128) : (const void*)scores, nb);
                }
            }
        }
        cp_async_commit();          // a group per step, empty or not, keeps the wait count fixed
        fslot = (fslot == SG_RING - 1) ? 0 : fslot + 1;
        if (++fsub == SG_STEPS) { fsub = 0; fc += nwarp; }
    };
    fetch();
    fetch();
    int slot = 0;
    for (int64_t c = gwarp; c < nchunk; c += nwarp) {
        if (lane == 0) *s_mc = 0u;
        __syncwarp();
        uint32_t* bm_out = L.sure_bm + c * BMW;
        uint32_t n_sure = 0;                                          // lanes 0..15: set bits of the words they stored
#pragma unroll 1
        for (int sub = 0; sub < SG_STEPS; ++sub) {
            fetch();
            cp_async_wait<2>();                                       // this lane's pieces of the step have landed ...
            __syncwarp();                                             // ... and so have the other lanes'
            const uint32_t* step_s = s_ring + slot * SG_STEP;
            const int64_t i0 = c * SG_CH + sub * SG_STEP;
#pragma unroll
            for (int sl = 0; sl < SG_STEP / 32; ++sl) {
                const uint32_t r = step_s[sl * 32 + lane];
                bool sure, cand;
                if (MODE == 2) {
                    cand = true; sure = order_key(r) > hi;
                } else {
                    const uint32_t sv = (MODE == 0) ? r : (r ^ ((uint32_t)((int32_t)r >> 31) & 0x7FFFFFFFu));
                    cand = sv - lo_s <= range;
                    sure = cand && (int32_t)sv > (int32_t)hi_s;
                }
                const uint32_t bs = __ballot_sync(0xFFFFFFFFu, sure), bc = __ballot_sync(0xFFFFFFFFu, cand);
                if (lane == 0) { s_w[sl] = bs; s_w[16 + sl] = bc; }   // the slot's words of the two bitmaps
            }
            __syncwarp();
            uint32_t w_sure = 0, w_may = 0;                           // lane s < 16: the two bitmap words of slot s
            if (lane < SG_STEP / 32) { w_sure = s_w[lane]; w_may = s_w[16 + lane] & ~w_sure; }
            if (N - i0 < SG_STEP) {                                   // ragged end: drop what lies beyond N
                const int64_t left = N - (i0 + lane * 32);            // scores of slot `lane` that exist
                const uint32_t valid = left >= 32 ? 0xFFFFFFFFu : (left > 0 ? (1u << (int)left) - 1u : 0u);
                w_sure &= valid; w_may &= valid;
            }
            if (lane < SG_STEP / 32) { bm_out[sub * (SG_STEP / 32) + lane] = w_sure; n_sure += (uint32_t)__popc(w_sure); }
            // second class: lane L takes half L & 1 of word L >> 1
            uint32_t half = (__shfl_sync(0xFFFFFFFFu, w_may, lane >> 1) >> ((lane & 1) * 16)) & 0xFFFFu;
            while (half) {
                const int b = __ffs((int)half) - 1;
                half &= half - 1u;
                const uint32_t idx = (uint32_t)(lane * 16 + b);       // score of the step
                const uint32_t r = step_s[idx];
                const uint32_t key = (MODE == 0) ? (r | 0x80000000u) : order_key(r);
                const uint32_t slot_m = atomicAdd(s_mc, 1u);          // pairs: any order
                *L.key(c, slot_m) = key;
                *L.off(c, slot_m) = (uint16_t)(sub * SG_STEP + idx);
                atomicAdd(&s_h[(key - lo) >> sh1], 1u);
            }
            __syncwarp();                                             // every lane is done with the step before its slot is refilled
            slot = (slot == SG_RING - 1) ? 0 : slot + 1;
        }
        n_sure = __reduce_add_sync(0xFFFFFFFFu, n_sure);
        if (lane == 0) {
            const uint32_t m = *s_mc;
            chunk_cnt[c] = n_sure | (m << 16);
            sure_total += n_sure; maybe_total += m;
        }
        __syncwarp();
    }
    cp_async_wait<0>();
}

__global__ void __launch_bounds__(SG_T, 4)
select_gather_kernel(const float* __restrict__ scores, int64_t N, int64_t k, BracketState* __restrict__ bs,
                     const ChunkLists L, uint32_t* __restrict__ chunk_cnt, uint32_t* __restrict__ hist1)
{
    dep_wait();
    dep_release();
    extern __shared__ __align__(16) uint8_t s_dyn[];      // per warp: ring of SG_RING steps of raw scores
    __shared__ uint32_t s_h[B1_BINS];
    __shared__ uint32_t s_mc[SG_T / 32];
    __shared__ uint32_t s_bw[SG_T / 32][32];
    const int tid = threadIdx.x;
    for (int i = tid; i < B1_BINS; i += SG_T) s_h[i] = 0;
    __syncthreads();
    const uint32_t lo = bs->lo_key, hi = bs->hi_key, sh1 = bs->sh[0];
    unsigned long long sure_total = 0, maybe_total = 0;
    uint32_t* s_ring = reinterpret_cast<uint32_t*>(s_dyn) + (tid >> 5) * (SG_RING * SG_STEP);
    if (lo > 0x80000000u) gather_chunks<0>(scores, N, lo, hi, sh1, L, chunk_cnt, s_h, &s_mc[tid >> 5], s_bw[tid >> 5], s_ring, sure_total, maybe_total);
    else if (lo > 0u) gather_chunks<1>(scores, N, lo, hi, sh1, L, chunk_cnt, s_h, &s_mc[tid >> 5], s_bw[tid >> 5], s_ring, sure_total, maybe_total);
    else gather_chunks<2>(scores, N, lo, hi, sh1, L, chunk_cnt, s_h, &s_mc[tid >> 5], s_bw[tid >> 5], s_ring, sure_total, maybe_total);
    __syncthreads();
    for (int i = tid; i < B1_BINS; i += SG_T)
        if (s_h[i]) atomicAdd(&hist1[i], s_h[i]);
    if ((tid & 31) == 0) {
        if (sure_total) atomicAdd(&bs->n_sure, sure_total);
        if (maybe_total) atomicAdd(&bs->n_maybe, maybe_total);
    }
    if (!last_block_done(&bs->ticket[2])) return;
    // the last block: is T inside the bracket? then the first radix round on key - lo
    const unsigned long long n_sure = *reinterpret_cast<volatile unsigned long long*>(&bs->n_sure);
    const unsigned long long n_maybe = *reinterpret_cast<volatile unsigned long long*>(&bs->n_maybe);
    const bool inside = n_sure < (unsigned long long)k && (unsigned long long)k <= n_sure + n_maybe;
    uint32_t bin = 0; int64_t krem = 0;
    const bool found = inside && block_find_bin<B1_BINS>(hist1, k - (int64_t)n_sure, &bin, &krem);
    if (tid == 0) {
        if (found) { bs->rel_prefix = bin; bs->k_rem = krem; bs->T = lo + (bin << sh1); }
        else bs->fallback = 1u;
    }
}

// Radix rounds 2 and 3 on the pairs: keys whose higher bits of key - lo equal the prefix fixed so far are
// histogrammed on the round's bits; the last block to finish fixes them. A round of zero bits does nothing.
template <int ROUND>
__device__ __forceinline__ void pair_hist_body(const ChunkLists& L, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk,
                                               BracketState* __restrict__ bs, uint32_t* __restrict__ hist)
{
    __shared__ uint32_t s_h[B23_BINS];
    const uint32_t b = bs->b[ROUND];
    if (b == 0u) return;
    for (int i = threadIdx.x; i < B23_BINS; i += SG_T) s_h[i] = 0;
    __syncthreads();
    const uint32_t lo = bs->lo_key, prefix = bs->rel_prefix, sh_prev = bs->sh[ROUND - 1], sh = bs->sh[ROUND], mask = (1u << b) - 1u;
    const int lane = threadIdx.x & 31;
    const int64_t nwarp = (int64_t)gridDim.x * (SG_T / 32);
    auto add = [&](uint32_t key) {
        const uint32_t rel = key - lo;
        if ((rel >> sh_prev) == prefix) atomicAdd(&s_h[(rel >> sh) & mask], 1u);
    };
    // a warp takes PG consecutive chunks at a time: their counts in one load, then the first 128 pairs of every one
    // of them in flight together (a chunk holds some 90 pairs; a list is too short to hide a memory round trip)
    for (int64_t c0 = ((int64_t)blockIdx.x * (SG_T / 32) + (threadIdx.x >> 5)) * PG; c0 < nchunk; c0 += nwarp * PG) {
        const int nc = (int)((nchunk - c0 < PG) ? nchunk - c0 : PG);
        const uint32_t cnt_l = (lane < nc) ? __ldg(chunk_cnt + c0 + lane) >> 16 : 0u;
        uint32_t v[PG][PU];
#pragma unroll
        for (int q = 0; q < PG; ++q) {
            const int m = (int)__shfl_sync(0xFFFFFFFFu, cnt_l, q);
            const uint32_t* seg = L.key_p + (c0 + q) * PP;
#pragma unroll
            for (int t = 0; t < PU; ++t) v[q][t] = (lane + 32 * t < m) ? __ldg(seg + lane + 32 * t) : 0u;
        }
#pragma unroll
        for (int q = 0; q < PG; ++q) {
            const int m = (int)__shfl_sync(0xFFFFFFFFu, cnt_l, q);
#pragma unroll
            for (int t = 0; t < PU; ++t) if (lane + 32 * t < m) add(v[q][t]);
            if (m > PP) {
                const uint32_t* seg = L.key_o + (c0 + q) * SG_CH;
                for (int j = PP + lane; j < m; j += 32) add(__ldg(seg + j));
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < B23_BINS; i += SG_T)
        if (s_h[i]) atomicAdd(&hist[i], s_h[i]);
    if (!last_block_done(&bs->ticket[2 + ROUND])) return;
    uint32_t bin = 0; int64_t krem = 0;
    const bool found = block_find_bin<B23_BINS>(hist, bs->k_rem, &bin, &krem);
    if (threadIdx.x == 0) {
        if (found) { const uint32_t np = (prefix << b) | bin; bs->rel_prefix = np; bs->k_rem = krem; bs->T = lo + (np << sh); }
        else bs->fallback = 1u;          // cannot happen for counts that are consistent; fail safe
    }
}

// Per chunk: how many of its scores are larger than T (the first class, counted by the streaming pass, and the pairs above T) and how many equal
// T. Block b owns the chunks [b R, (b + 1) R) and leaves their totals for the write kernel.
__device__ __forceinline__ void pair_count_body(const ChunkLists& L, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk, int64_t R,
                                                int64_t G, const BracketState* __restrict__ bs, int32_t* __restrict__ blk_cnt,
                                                int64_t* __restrict__ blk_tot)
{
    __shared__ int64_t s_t[2][SG_T / 32];
    if ((int64_t)blockIdx.x >= G) return;            // the launch may be wider than the partition
    const uint32_t T = bs->T;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c_lo = (int64_t)blockIdx.x * R, c_hi = (c_lo + R < nchunk) ? c_lo + R : nchunk;
    int64_t tot_gt = 0, tot_eq = 0;
    for (int64_t c0 = c_lo + warp * PG; c0 < c_hi; c0 += (SG_T / 32) * PG) {
        const int nc = (int)((c_hi - c0 < PG) ? c_hi - c0 : PG);
        const uint32_t cw = (lane < nc) ? __ldg(chunk_cnt + c0 + lane) : 0u;
        uint32_t v[PG][PU];
#pragma unroll
        for (int q = 0; q < PG; ++q) {
            const int m = (int)(__shfl_sync(0xFFFFFFFFu, cw, q) >> 16);
            const uint32_t* seg = L.key_p + (c0 + q) * PP;
#pragma unroll
            for (int t = 0; t < PU; ++t) v[q][t] = (lane + 32 * t < m) ? __ldg(seg + lane + 32 * t) : 0u;
        }
        int my_gt = 0, my_eq = 0;                   // lane q ends up with the counts of chunk c0 + q
#pragma unroll
        for (int q = 0; q < PG; ++q) {
            const uint32_t w = __shfl_sync(0xFFFFFFFFu, cw, q);
            const int n = (int)(w & 0xFFFFu), m = (int)(w >> 16);
            int gt = 0, eq = 0;
#pragma unroll
            for (int t = 0; t < PU; ++t) if (lane + 32 * t < m) { gt += (v[q][t] > T); eq += (v[q][t] == T); }
            if (m > PP) {
                const uint32_t* seg = L.key_o + (c0 + q) * SG_CH;
                for (int j = PP + lane; j < m; j += 32) { const uint32_t key = __ldg(seg + j); gt += (key > T); eq += (key == T); }
            }
            gt = __reduce_add_sync(0xFFFFFFFFu, gt);
            eq = __reduce_add_sync(0xFFFFFFFFu, eq);
            if (lane == q) { my_gt = gt + n; my_eq = eq; }      // n: the chunk's scores above hi
        }
        if (lane < nc) *reinterpret_cast<int2*>(blk_cnt + 2 * (c0 + lane)) = make_int2(my_gt, my_eq);
        tot_gt += my_gt; tot_eq += my_eq;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { tot_gt += __shfl_xor_sync(0xFFFFFFFFu, tot_gt, o); tot_eq += __shfl_xor_sync(0xFFFFFFFFu, tot_eq, o); }
    if (lane == 0) { s_t[0][warp] = tot_gt; s_t[1][warp] = tot_eq; }
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t a = 0, b = 0;
        for (int w = 0; w < SG_T / 32; ++w) { a += s_t[0][w]; b += s_t[1][w]; }
        blk_tot[2 * blockIdx.x] = a; blk_tot[2 * blockIdx.x + 1] = b;
    }
}

// Final write. Block b owns the chunks [b R, (b + 1) R) (the partition of the count kernel), its warps consecutive
// runs of them. For a chunk the warp marks, in a 4096-bit map in shared memory, the offsets of the pairs that are
// selected: key above T, or equal to T while ties are still admitted (ties by ascending offset, ranked through a
// second map if the chunk holds the last admitted tie). OR-ed with the chunk's first-class bitmap this is the bitmap
// of the selected scores; a lane owns four of its words, a warp scan of their population counts gives the lane its
// place in the output, and it writes the indices of its set bits in ascending order.
__device__ __forceinline__ void pair_write_body(const ChunkLists& L, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk, int64_t R,
                                                int64_t G, const BracketState* __restrict__ bs, const int32_t* __restrict__ blk_cnt,
                                                const int64_t* __restrict__ blk_tot, int64_t* __restrict__ indices)
{
    __shared__ __align__(16) uint32_t s_bm[SG_T / 32][2][BMW];
    __shared__ uint16_t s_stage[SG_T / 32][SG_CH / 4];
    __shared__ int64_t s_w[2][SG_T / 32];
    if ((int64_t)blockIdx.x >= G) return;            // the launch may be wider than the partition
    const uint32_t T = bs->T;
    const int64_t k_ties = bs->k_rem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint16_t* stage = s_stage[warp];
    int64_t gt_run, eq_run;
    block_base_before(blk_tot, gt_run, eq_run);
    const int64_t c_lo = (int64_t)blockIdx.x * R, c_hi = (c_lo + R < nchunk) ? c_lo + R : nchunk;
    // this warp's run of chunks, and what the warps before it in the block contribute
    const int64_t per_w = (c_hi - c_lo + SG_T / 32 - 1) / (SG_T / 32);
    const int64_t w_lo = (c_lo + warp * per_w < c_hi) ? c_lo + warp * per_w : c_hi;
    const int64_t w_hi = (w_lo + per_w < c_hi) ? w_lo + per_w : c_hi;
    {
        int64_t a = 0, b = 0;
        for (int64_t c = w_lo + lane; c < w_hi; c += 32) { const int2 v = *reinterpret_cast<const int2*>(blk_cnt + 2 * c); a += v.x; b += v.y; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { a += __shfl_xor_sync(0xFFFFFFFFu, a, o); b += __shfl_xor_sync(0xFFFFFFFFu, b, o); }
        if (lane == 0) { s_w[0][warp] = a; s_w[1][warp] = b; }
        __syncthreads();
        for (int w = 0; w < warp; ++w) { gt_run += s_w[0][w]; eq_run += s_w[1][w]; }
    }
    uint32_t* bm_sel = s_bm[warp][0];
    uint32_t* bm_tie = s_bm[warp][1];
    static_assert(BMW == 128, "a lane owns four bitmap words");
    // everything the next chunk needs is requested while the current one is worked on
    uint32_t cw_n = 0; int2 ge_n = make_int2(0, 0); uint4 sure_n = make_uint4(0u, 0u, 0u, 0u);
    uint32_t pk_n[PU], po_n[PU];
    auto request = [&](int64_t c) {
        cw_n = __ldg(chunk_cnt + c);
        ge_n = *reinterpret_cast<const int2*>(blk_cnt + 2 * c);
        sure_n = __ldg(reinterpret_cast<const uint4*>(L.sure_bm + c * BMW) + lane);
        // the first PP pairs: slots beyond the chunk's count hold stale data and are ignored below
#pragma unroll
        for (int t = 0; t < PU; ++t) { pk_n[t] = __ldg(L.key_p + c * PP + lane + 32 * t); po_n[t] = (uint32_t)__ldg(L.off_p + c * PP + lane + 32 * t); }
    };
    if (w_lo < w_hi) request(w_lo);
    for (int64_t c = w_lo; c < w_hi; ++c) {
        const uint32_t cw = cw_n;
        const int2 ge = ge_n;
        uint4 f4 = sure_n;
        uint32_t pk[PU], po[PU];
#pragma unroll
        for (int t = 0; t < PU; ++t) { pk[t] = pk_n[t]; po[t] = po_n[t]; }
        if (c + 1 < w_hi) request(c + 1);
        const int m = (int)(cw >> 16);
        if (m > 0) {
            reinterpret_cast<uint4*>(bm_sel)[lane] = make_uint4(0u, 0u, 0u, 0u);
            reinterpret_cast<uint4*>(bm_tie)[lane] = make_uint4(0u, 0u, 0u, 0u);
            __syncwarp();
#pragma unroll
            for (int t = 0; t < PU; ++t)
                if (lane + 32 * t < m && pk[t] >= T) atomicOr((pk[t] > T ? bm_sel : bm_tie) + (po[t] >> 5), 1u << (po[t] & 31u));
            for (int j = PP + lane; j < m; j += 32) {
                const uint32_t key = __ldg(L.key_o + c * SG_CH + j);
                if (key >= T) { const uint32_t o = __ldg(L.off_o + c * SG_CH + j); atomicOr((key > T ? bm_sel : bm_tie) + (o >> 5), 1u << (o & 31u)); }
            }
            __syncwarp();
            uint4 s4 = reinterpret_cast<const uint4*>(bm_sel)[lane];
            if (ge.y > 0) {
                const int64_t room64 = k_ties - eq_run;                               // ties this chunk may still admit
                const uint4 t4 = reinterpret_cast<const uint4*>(bm_tie)[lane];
                if (room64 >= (int64_t)ge.y) {                                        // all of them
                    s4.x |= t4.x; s4.y |= t4.y; s4.z |= t4.z; s4.w |= t4.w;
                } else if (room64 > 0) {                                              // the first room64 by offset
                    const uint32_t tw[4] = {t4.x, t4.y, t4.z, t4.w};
                    const int cnt = __popc(tw[0]) + __popc(tw[1]) + __popc(tw[2]) + __popc(tw[3]);
                    int incl = cnt;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) { const int a = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += a; }
                    int rank = incl - cnt;                                            // ties before this lane's words
                    const int room = (int)room64;
                    uint32_t keep[4];
                    for (int q = 0; q < 4; ++q) {
                        uint32_t word = tw[q];
                        keep[q] = 0u;
                        while (word && rank < room) { const uint32_t low = word & (0u - word); keep[q] |= low; word ^= low; ++rank; }
                        rank += __popc(word);
                    }
                    s4.x |= keep[0]; s4.y |= keep[1]; s4.z |= keep[2]; s4.w |= keep[3];
                }
            }
            f4.x |= s4.x; f4.y |= s4.y; f4.z |= s4.z; f4.w |= s4.w;
            __syncwarp();       // the maps are read: they may be cleared for the next chunk
        }
        // The selected scores of the chunk, in index order: a lane's four words cover offsets [128 lane, 128 lane + 128); a
        // warp scan of the lanes' population counts ranks their set bits, which are staged as 16-bit offsets and then
        // leave as consecutive 64-bit indices, 32 per store (a lane writing its own indices one by one touched a
        // 32-byte sector per 8 bytes written). The staging area holds a quarter of a chunk; a chunk with more selected
        // scores than that goes through it quarter by quarter.
        int64_t* out = indices + gt_run + (eq_run < k_ties ? eq_run : k_ties);
        const int64_t ibase = c * SG_CH;
        {
            const uint32_t fw[4] = {f4.x, f4.y, f4.z, f4.w};
            const int pc[4] = {__popc(fw[0]), __popc(fw[1]), __popc(fw[2]), __popc(fw[3])};
            const int cnt = pc[0] + pc[1] + pc[2] + pc[3];
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int a = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += a; }
            const int tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (tot <= SG_CH / 4) {
                int pos = incl - cnt;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    // a word's bits from the top down into the end of its run: one leading-zero count per bit
                    // (bit scans run on the quarter-rate unit; finding the lowest bit takes two of them)
                    uint32_t word = fw[q];
                    const uint32_t obase = (uint32_t)(lane * 128 + q * 32);
                    pos += pc[q];
                    int pe = pos;
                    while (word) {
                        const int b = 31 - __clz((int)word);
                        word ^= 1u << b;
                        stage[--pe] = (uint16_t)(obase + (uint32_t)b);
                    }
                }
                __syncwarp();
                for (int i = lane; i < tot; i += 32) out[i] = ibase + stage[i];
                __syncwarp();       // the staging area is rewritten by the next chunk
                gt_run += ge.x; eq_run += ge.y;
                continue;
            }
        }
        reinterpret_cast<uint4*>(bm_sel)[lane] = f4;
        __syncwarp();
#pragma unroll 1
        for (int qt = 0; qt < 4; ++qt) {
            uint32_t word = bm_sel[qt * 32 + lane];
            const int cnt = __popc(word);
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int a = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += a; }
            const int tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (tot == 0) continue;
            int pos = incl - cnt;
            const uint32_t obase = (uint32_t)((qt * 32 + lane) * 32);
            while (word) {
                const int b = __ffs((int)word) - 1;
                word &= word - 1u;
                stage[pos++] = (uint16_t)(obase + (uint32_t)b);
            }
            __syncwarp();
            for (int i = lane; i < tot; i += 32) out[i] = ibase + stage[i];
            out += tot;
            __syncwarp();       // the staging area is rewritten by the next quarter
        }
        gt_run += ge.x; eq_run += ge.y;
    }
}

// The launches behind the streaming pass. Each does its step of the bracketed path or, if the bracket missed T (the
// flag the streaming pass left), the matching step of the exact multi-pass path on the scores: one launch serves
// both, so that the rare path costs one extra launch (its final write) instead of five that return at once.
struct FallbackArgs {
    const float* scores; int64_t N, k;
    SelectState* state; uint32_t* hist;          // three cleared histograms
    int64_t nblk, R, G;                          // units of 2048 scores and their partition over blocks
};

__global__ void __launch_bounds__(SG_T)
bracket_round2_kernel(const ChunkLists L, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk, BracketState* __restrict__ bs,
                      uint32_t* __restrict__ hist, const FallbackArgs fb)
{
    dep_wait();
    dep_release();
    if (bs->fallback != 0u) select_hist_body<0>(fb.scores, fb.N, fb.k, fb.state, fb.hist);
    else pair_hist_body<1>(L, chunk_cnt, nchunk, bs, hist);
}
__global__ void __launch_bounds__(SG_T)
bracket_round3_kernel(const ChunkLists L, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk, BracketState* __restrict__ bs,
                      uint32_t* __restrict__ hist, const FallbackArgs fb)
{
    dep_wait();
    dep_release();
    if (bs->fallback != 0u) select_hist_body<1>(fb.scores, fb.N, fb.k, fb.state, fb.hist + 2048);
    else pair_hist_body<2>(L, chunk_cnt, nchunk, bs, hist);
}
__global__ void __launch_bounds__(SG_T)
bracket_count_kernel(const ChunkLists L, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk, int64_t R, int64_t G,
                     const BracketState* __restrict__ bs, int32_t* __restrict__ blk_cnt, int64_t* __restrict__ blk_tot,
                     const FallbackArgs fb)
{
    dep_wait();
    dep_release();
    if (bs->fallback != 0u) select_hist_body<2>(fb.scores, fb.N, fb.k, fb.state, fb.hist + 4096);
    else pair_count_body(L, chunk_cnt, nchunk, R, G, bs, blk_cnt, blk_tot);
}
__global__ void __launch_bounds__(SG_T, 6)
bracket_write_kernel(const ChunkLists L, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk, int64_t R, int64_t G,
                     const BracketState* __restrict__ bs, int32_t* __restrict__ blk_cnt, int64_t* __restrict__ blk_tot,
                     int64_t* __restrict__ indices, const FallbackArgs fb)
{
    dep_wait();
    dep_release();
    if (bs->fallback != 0u) select_count_body(fb.scores, fb.N, fb.nblk, fb.R, fb.G, fb.state, blk_cnt, blk_tot);
    else pair_write_body(L, chunk_cnt, nchunk, R, G, bs, blk_cnt, blk_tot, indices);
}

// ------------------------------------------------------------------------------------------------
// Small N (every workload of the paper): one thread-block cluster of eight CTAs does the whole selection
// in one launch. Each CTA loads its contiguous slice of the scores once and keeps the keys in shared
// memory; the three radix rounds build per-CTA histograms there and every CTA sums the eight histograms
// through distributed shared memory; the slice totals of {key > T}, {key == T} are exchanged the same way
// and each CTA writes its part of the answer in index order. One read of the scores, no workspace, and the
// only waits are the hardware cluster barrier.
// ------------------------------------------------------------------------------------------------
constexpr int CL_CTAS = 8;
constexpr int CL_T = 1024;
constexpr int CL_CAP = 45056;                              // keys per CTA held in shared memory (176 KiB)
constexpr int64_t CL_MAX_N = (int64_t)CL_CTAS * CL_CAP;    // 360 448 scores

__device__ __forceinline__ uint32_t ld_dsmem_u32(uint32_t cluster_addr)
{
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
    return v;
}

__global__ void __cluster_dims__(CL_CTAS, 1, 1) __launch_bounds__(CL_T, 1)
select_cluster_kernel(const float* __restrict__ scores, int64_t N, int64_t k, int64_t* __restrict__ indices)
{
    extern __shared__ uint32_t s_key[];                    // [CL_CAP] keys of this CTA's slice
    __shared__ uint32_t s_hist2[2][2048];                  // alternating per round: one cluster barrier per round suffices
    __shared__ int64_t s_w[2][32];
    __shared__ uint32_t s_bin;
    __shared__ int64_t s_krem;
    __shared__ int s_tot[2];                               // this slice's counts of {key > T}, {key == T}
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = tc::cluster_ctarank();
    const int64_t per = ((N + CL_CTAS - 1) / CL_CTAS + 3) & ~(int64_t)3;          // slice length, a multiple of 4
    const int64_t i0 = (int64_t)rank * per;
    const int n_loc = (int)((i0 >= N) ? 0 : ((N - i0 < per) ? N - i0 : per));
    for (int i = tid; i < n_loc; i += CL_T) s_key[i] = order_key(__float_as_uint(__ldg(scores + i0 + i)));
    __syncthreads();

    uint32_t prefix = 0;
    int64_t k_rem = k;
#pragma unroll 1
    for (int round = 0; round < 3; ++round) {
        const int shift = (round == 0) ? 21 : (round == 1) ? 10 : 0;
        const int bits = (round == 2) ? 10 : 11;
        const uint32_t mask = (1u << bits) - 1u;
        uint32_t* s_hist = s_hist2[round & 1];
        for (int i = tid; i < 2048; i += CL_T) s_hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < n_loc; i += CL_T) {
            const uint32_t key = s_key[i];
            if (round == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&s_hist[(key >> shift) & mask], 1u);
        }
        __syncthreads();
        tc::cluster_sync_all();                           // all eight histograms of this round complete
        // every CTA sums the eight histograms and finds the bin of the k_rem-th largest key: thread t owns, from the
        // top, bins 2047-2t and 2046-2t (rounds 0, 1) or bin 1023-t (round 2)
        const int nb = 1 << bits;
        const int per_t = nb / CL_T;                      // 2 or 1
        int64_t c[2] = {0, 0};
        for (int u = 0; u < per_t; ++u) {
            const int b = nb - 1 - (tid * per_t + u);
            const uint32_t own = tc::smem_u32(&s_hist[b]);
            int64_t sum = 0;
#pragma unroll
            for (uint32_t r = 0; r < CL_CTAS; ++r) sum += ld_dsmem_u32(tc::map_to_cta(own, r));
            c[u] = sum;
        }
        const int64_t mine = c[0] + c[1];
        int64_t inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int64_t a = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= o) inc += a;
        }
        if (lane == 31) s_w[0][warp] = inc;
        __syncthreads();
        int64_t pre = inc - mine;
        for (int w = 0; w < warp; ++w) pre += s_w[0][w];
        for (int u = 0; u < per_t; ++u) {
            if (pre < k_rem && k_rem <= pre + c[u]) { s_bin = (uint32_t)(nb - 1 - (tid * per_t + u)); s_krem = k_rem - pre; }
            pre += c[u];
        }
        __syncthreads();
        prefix = (prefix << bits) | s_bin;
        k_rem = s_krem;
        // no barrier here: the next round fills the other histogram buffer, and this one is cleared again only after
        // the next round's cluster barrier, which every CTA reaches after it has finished reading it
    }
    const uint32_t T = prefix;
    const int64_t k_ties = k_rem;

    // thread t owns a run of consecutive keys of the slice (odd length: no shared-memory bank conflicts)
    const int len = ((n_loc + CL_T - 1) / CL_T) | 1;
    const int j0 = tid * len, j1 = (j0 + len < n_loc) ? j0 + len : n_loc;
    int gt = 0, eq = 0;
    for (int j = j0; j < j1; ++j) { const uint32_t key = s_key[j]; gt += (key > T); eq += (key == T); }
    int ig = gt, ie = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xFFFFFFFFu, ig, o), b = __shfl_up_sync(0xFFFFFFFFu, ie, o);
        if (lane >= o) { ig += a; ie += b; }
    }
    if (lane == 31) { s_w[0][warp] = ig; s_w[1][warp] = ie; }
    __syncthreads();
    int64_t gt_before = ig - gt, eq_before = ie - eq;
    for (int w = 0; w < warp; ++w) { gt_before += s_w[0][w]; eq_before += s_w[1][w]; }
    if (tid == CL_T - 1) { s_tot[0] = (int)(gt_before + gt); s_tot[1] = (int)(eq_before + eq); }
    __syncthreads();
    tc::cluster_sync_all();                               // slice totals visible to the other CTAs
    for (uint32_t r = 0; r < rank; ++r) {
        gt_before += (int)ld_dsmem_u32(tc::map_to_cta(tc::smem_u32(&s_tot[0]), r));
        eq_before += (int)ld_dsmem_u32(tc::map_to_cta(tc::smem_u32(&s_tot[1]), r));
    }
    for (int j = j0; j < j1; ++j) {
        const uint32_t key = s_key[j];
        const bool g = key > T, e = key == T;
        if (g || (e && eq_before < k_ties)) indices[gt_before + (eq_before < k_ties ? eq_before : k_ties)] = i0 + j;
        gt_before += g; eq_before += e;
    }
    tc::cluster_sync_all();                               // no CTA leaves while another may still read its shared memory
}

SelectWs carve(void* ws, int64_t N)
{
    SelectWs w;
    uint8_t* p = reinterpret_cast<uint8_t*>(ws);
    w.hist = reinterpret_cast<uint32_t*>(p); p += 3 * 2048 * sizeof(uint32_t);
    w.state = reinterpret_cast<SelectState*>(p); p += 256;
    w.blk_tot = reinterpret_cast<int64_t*>(p); p += (size_t)SEL_MAX_GRID * 2 * sizeof(int64_t);
    w.blk_cnt = reinterpret_cast<int32_t*>(p);
    (void)N;
    return w;
}

size_t compact_workspace_bytes(int64_t N)
{
    const int64_t nblk = sel_nblk(N > 0 ? N : 1);
    return 3 * 2048 * sizeof(uint32_t) + 256 + (size_t)SEL_MAX_GRID * 2 * sizeof(int64_t) +
           align_up((size_t)nblk * 2 * sizeof(int32_t), 256);
}

BracketWs carve_bracket(void* ws, int64_t N)
{
    BracketWs w;
    uint8_t* p = reinterpret_cast<uint8_t*>(ws);
    w.hist = reinterpret_cast<uint32_t*>(p); p += (size_t)BR_HIST_WORDS * sizeof(uint32_t);
    w.bstate = reinterpret_cast<BracketState*>(p); p += 256;
    w.fstate = reinterpret_cast<SelectState*>(p); p += 256;
    const int64_t nblk = sel_nblk(N), nchunk = sg_nchunk(N);
    w.blk_tot = reinterpret_cast<int64_t*>(p); p += (size_t)SEL_MAX_GRID * 2 * sizeof(int64_t);
    w.blk_cnt = reinterpret_cast<int32_t*>(p); p += align_up((size_t)nblk * 2 * sizeof(int32_t), 256);
    w.sample_key = reinterpret_cast<uint32_t*>(p); p += SG_SAMPLE * sizeof(uint32_t);
    w.chunk_cnt = reinterpret_cast<uint32_t*>(p); p += align_up((size_t)nchunk * sizeof(uint32_t), 256);
    w.L.sure_bm = reinterpret_cast<uint32_t*>(p); p += align_up((size_t)nchunk * BMW * sizeof(uint32_t), 256);
    w.L.key_p = reinterpret_cast<uint32_t*>(p); p += align_up((size_t)nchunk * PP * sizeof(uint32_t), 256);
    w.L.off_p = reinterpret_cast<uint16_t*>(p); p += align_up((size_t)nchunk * PP * sizeof(uint16_t), 256);
    w.L.off_o = reinterpret_cast<uint16_t*>(p); p += align_up((size_t)nchunk * SG_CH * sizeof(uint16_t), 256);
    w.L.key_o = reinterpret_cast<uint32_t*>(p);
    return w;
}

size_t bracket_workspace_bytes(int64_t N)
{
    const int64_t nblk = sel_nblk(N), nchunk = sg_nchunk(N);
    return (size_t)BR_HIST_WORDS * sizeof(uint32_t) + 512 + (size_t)SEL_MAX_GRID * 2 * sizeof(int64_t) +
           align_up((size_t)nblk * 2 * sizeof(int32_t), 256) + SG_SAMPLE * sizeof(uint32_t) +
           align_up((size_t)nchunk * sizeof(uint32_t), 256) + align_up((size_t)nchunk * BMW * sizeof(uint32_t), 256) +
           align_up((size_t)nchunk * PP * sizeof(uint32_t), 256) + align_up((size_t)nchunk * PP * sizeof(uint16_t), 256) +
           align_up((size_t)nchunk * SG_CH * sizeof(uint16_t), 256) + (size_t)nchunk * SG_CH * sizeof(uint32_t);
}
static_assert(sizeof(BracketState) <= 256 && sizeof(SelectState) <= 256, "state regions are 256 bytes");

// The exact multi-pass path on the scores themselves (five reads, five launches). hist: three cleared histograms;
// state: cleared.
cudaError_t launch_multipass(const float* scores, int64_t N, int64_t k, int64_t* indices, uint32_t* hist,
                             SelectState* state, int32_t* blk_cnt, int64_t* blk_tot, cudaStream_t st)
{
    int64_t hb = (N / 4 + SEL_T - 1) / SEL_T;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (hb > cap) hb = cap;
    if (hb < 1) hb = 1;
    const int64_t nblk = sel_nblk(N);
    const int64_t G = nblk < SEL_MAX_GRID ? nblk : SEL_MAX_GRID;
    const int64_t R = (nblk + G - 1) / G;
    cudaError_t e;
    if ((e = launch_after(select_hist_kernel<0>, (unsigned)hb, SEL_T, 0, st, scores, N, k, state, hist)) != cudaSuccess) return e;
    if ((e = launch_after(select_hist_kernel<1>, (unsigned)hb, SEL_T, 0, st, scores, N, k, state, hist + 2048)) != cudaSuccess) return e;
    if ((e = launch_after(select_hist_kernel<2>, (unsigned)hb, SEL_T, 0, st, scores, N, k, state, hist + 4096)) != cudaSuccess) return e;
    if ((e = launch_after(select_count_kernel, (unsigned)G, SEL_T, 0, st, scores, N, nblk, R, G, state, blk_cnt, blk_tot)) != cudaSuccess) return e;
    if ((e = launch_after(select_write_kernel, (unsigned)G, SEL_T, 0, st, scores, N, nblk, R, state, blk_cnt, blk_tot, indices, Gate{nullptr, 0u})) != cudaSuccess) return e;
    count_launches(5);
    return cudaGetLastError();
}

cudaError_t launch_bracketed(const float* scores, int64_t N, int64_t k, int64_t* indices, void* ws, bool force_short,
                             cudaStream_t st)
{
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(select_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (SG_T / 32) * SG_RING * SG_STEP * (int)sizeof(uint32_t));
    });
    if (attr_err != cudaSuccess) return attr_err;
    BracketWs w = carve_bracket(ws, N);
    const int64_t nchunk = sg_nchunk(N);
    const int64_t gcap = (int64_t)sm_count() * 4;          // the gather kernel's resident blocks (48 KiB ring each)
    const int64_t gneed = (nchunk + SG_T / 32 - 1) / (SG_T / 32);       // a warp per chunk
    const unsigned gb = (unsigned)(gneed < gcap ? gneed : gcap);
    const int64_t hneed = (nchunk + (SG_T / 32) * PG - 1) / ((SG_T / 32) * PG);     // a warp per PG chunks
    const int64_t hcap = (int64_t)sm_count() * 8;
    const int64_t hb = hneed < hcap ? hneed : hcap;
    // count and write: contiguous runs of chunks, every block resident at once (six per SM)
    int64_t G = (int64_t)sm_count() * 6;
    if (G > SEL_MAX_GRID) G = SEL_MAX_GRID;
    if (G > gneed) G = gneed;
    const int64_t R = (nchunk + G - 1) / G;
    uint32_t* hist1 = w.hist;
    uint32_t* hist2 = w.hist + B1_BINS;
    uint32_t* hist3 = hist2 + B23_BINS;
    uint32_t* hist_s = hist3 + B23_BINS + 3 * 2048;      // sample: first level, second level of lo, of hi
    // the exact multi-pass path, should the bracket miss: its grids, and its steps riding in the launches below
    FallbackArgs fb;
    fb.scores = scores; fb.N = N; fb.k = k; fb.state = w.fstate; fb.hist = hist3 + B23_BINS;
    fb.nblk = sel_nblk(N);
    fb.G = fb.nblk < SEL_MAX_GRID ? fb.nblk : SEL_MAX_GRID;
    fb.R = (fb.nblk + fb.G - 1) / fb.G;
    int64_t fhb = (N / 4 + SEL_T - 1) / SEL_T;
    if (fhb > hcap) fhb = hcap;
    const unsigned g_round = (unsigned)(hb > fhb ? hb : fhb), g_count = (unsigned)(G > fhb ? G : fhb), g_write = (unsigned)(G > fb.G ? G : fb.G);
    // histograms and both states are contiguous: one clear
    cudaError_t e = cudaMemsetAsync(w.hist, 0, (size_t)(BR_HIST_WORDS + 128) * sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    const size_t ring_bytes = (SG_T / 32) * SG_RING * SG_STEP * sizeof(uint32_t);
    const int fs = force_short ? 1 : 0;
    if ((e = launch_after(sample_level1_kernel, SS_BLOCKS, SEL_T, 0, st, scores, w.sample_key, N, k, w.bstate, hist_s)) != cudaSuccess) return e;
    if ((e = launch_after(sample_level2_kernel, SS_BLOCKS, SEL_T, 0, st, w.sample_key, N, k, w.bstate, hist_s + 4096, hist_s + 8192, fs)) != cudaSuccess) return e;
    if ((e = launch_after(select_gather_kernel, gb, SG_T, ring_bytes, st, scores, N, k, w.bstate, w.L, w.chunk_cnt, hist1)) != cudaSuccess) return e;
    if ((e = launch_after(bracket_round2_kernel, g_round, SG_T, 0, st, w.L, w.chunk_cnt, nchunk, w.bstate, hist2, fb)) != cudaSuccess) return e;
    if ((e = launch_after(bracket_round3_kernel, g_round, SG_T, 0, st, w.L, w.chunk_cnt, nchunk, w.bstate, hist3, fb)) != cudaSuccess) return e;
    if ((e = launch_after(bracket_count_kernel, g_count, SG_T, 0, st, w.L, w.chunk_cnt, nchunk, R, G, w.bstate, w.blk_cnt, w.blk_tot, fb)) != cudaSuccess) return e;
    if ((e = launch_after(bracket_write_kernel, g_write, SG_T, 0, st, w.L, w.chunk_cnt, nchunk, R, G, w.bstate, w.blk_cnt, w.blk_tot, indices, fb)) != cudaSuccess) return e;
    if ((e = launch_after(select_write_kernel, (unsigned)fb.G, SEL_T, 0, st, scores, N, fb.nblk, fb.R, w.fstate, w.blk_cnt, w.blk_tot, indices,
                          Gate{&w.bstate->fallback, 1u})) != cudaSuccess) return e;
    count_launches(8);
    return cudaGetLastError();
}

int g_select_path = 0;     // 0: by size; 1: multi-pass always; 2: bracketed with a bracket that is too high

}  // namespace

void set_select_path(int mode) { g_select_path = mode; }

static bool use_bracket(int64_t N) { return g_select_path != 1 && N > SG_MIN_N; }

size_t select_workspace_bytes(int64_t N)
{
    if (N > SG_MIN_N) return bracket_workspace_bytes(N);     // whatever the path chosen at launch time
    return compact_workspace_bytes(N);
}

cudaError_t launch_select_topk(const float* scores, int64_t N, int64_t k, int64_t* indices, void* ws,
                               cudaStream_t st)
{
    if (N == 0 || k == 0) return cudaSuccess;
    if (g_select_path != 1 && N <= CL_MAX_N) {
        static std::once_flag once;
        static cudaError_t attr_err = cudaSuccess;
        std::call_once(once, [] {
            attr_err = cudaFuncSetAttribute(select_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, CL_CAP * (int)sizeof(uint32_t));
        });
        if (attr_err != cudaSuccess) return attr_err;
        select_cluster_kernel<<<CL_CTAS, CL_T, CL_CAP * sizeof(uint32_t), st>>>(scores, N, k, indices);
        count_launches(1);
        return cudaGetLastError();
    }
    if (use_bracket(N)) return launch_bracketed(scores, N, k, indices, ws, g_select_path == 2, st);
    SelectWs w = carve(ws, N);
    cudaError_t e = cudaMemsetAsync(w.hist, 0, 3 * 2048 * sizeof(uint32_t) + 256, st);      // histograms and state
    if (e != cudaSuccess) return e;
    return launch_multipass(scores, N, k, indices, w.hist, w.state, w.blk_cnt, w.blk_tot, st);
}

}  // namespace qless

// ------------------------------------------------------------------------------------------------
// Selection without any allocation: the scratch of the radix select lives in a fixed device array.
// ------------------------------------------------------------------------------------------------

namespace qless {
namespace {

// 3 histograms (24 KiB) + state (256 B) + block totals (16 KiB) + counts of the MAX_N / 2048 = 2048 units
// (16 KiB) = 57 600 bytes; the array keeps its 74 KiB. Resident on every GPU that loads the library.
constexpr size_t kStaticScratchBytes = 74 * 1024;
static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of g_select_scratch on the current device. In host code the array's name only
// stands for the symbol; the address kernels can use has to be asked for, once per device.
qless_status static_scratch(void** out)
{
    int dev = 0;
    QLESS_CUDA_TRY(cudaGetDevice(&dev));
    QLESS_REQUIRE(dev >= 0 && dev < kMaxDevices, QLESS_ERR_UNSUPPORTED, "device ordinal %d beyond %d", dev, kMaxDevices);
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        QLESS_CUDA_TRY(cudaGetSymbolAddress(&p, g_select_scratch));
        QLESS_REQUIRE(p != nullptr, QLESS_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return QLESS_OK;
}

}  // namespace

}  // namespace qless

extern "C" qless_status qless_select_topk_static(const float* scores, int64_t N, double frac, int64_t* indices,
                                                 int64_t* k_out, void* cuda_stream)
{
    using namespace qless;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(N >= 0, QLESS_ERR_INVALID_ARG, "N must be >= 0");
    QLESS_REQUIRE(N <= (int64_t)QLESS_SELECT_STATIC_MAX_N, QLESS_ERR_UNSUPPORTED,
                  "qless_select_topk_static handles at most %d scores (N=%lld); use qless_select_topk with a workspace",
                  (int)QLESS_SELECT_STATIC_MAX_N, (long long)N);
    QLESS_REQUIRE(frac >= 0.0 && frac <= 1.0, QLESS_ERR_INVALID_ARG, "frac must be in [0, 1]");
    QLESS_REQUIRE(k_out != nullptr, QLESS_ERR_INVALID_ARG, "k_out (host) is required");
    double kf = std::floor(frac * (double)N + 1e-6);
    if (kf < 0.0) kf = 0.0;
    if (kf > (double)N) kf = (double)N;
    const int64_t k = (int64_t)kf;
    if (k > 0) {
        QLESS_REQUIRE(scores != nullptr && indices != nullptr, QLESS_ERR_INVALID_ARG, "scores and indices are required");
        QLESS_REQUIRE((reinterpret_cast<uintptr_t>(scores) % 16) == 0, QLESS_ERR_INVALID_ARG, "scores must be 16-byte aligned");
        static_assert(kStaticScratchBytes >= 3 * 2048 * 4 + 256 + SEL_MAX_GRID * 16 + 2048 * 8, "scratch array too small");
        QLESS_REQUIRE(select_workspace_bytes(N) <= kStaticScratchBytes, QLESS_ERR_UNSUPPORTED, "internal: scratch array too small");
    }
    *k_out = k;
    if (k == 0) return QLESS_OK;
    void* scratch = nullptr;
    qless_status s = static_scratch(&scratch);
    if (s != QLESS_OK) return s;
    // The histograms and the selection state are cleared inside; the block totals and the unit counts are
    // rewritten in full for this N before they are read, so nothing of the previous call's contents is used.
    QLESS_CUDA_TRY(launch_select_topk(scores, N, k, indices, scratch, st));
    return QLESS_OK;
}
