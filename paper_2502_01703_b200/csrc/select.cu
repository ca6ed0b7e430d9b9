// Stage 4: top-k by radix select on order-preserving 32-bit keys, then an index-ordered compaction.
// Three histogram passes (11 + 11 + 10 bits) fix the k-th largest key T exactly and the number of
// keys equal to T that are admitted (smallest indices first); the compaction writes the indices of
// {key > T} and of the admitted ties in ascending order.
#include <cmath>
#include <mutex>

#include "qless_kernels.h"
#include "tc_common.cuh"

namespace qless {

namespace {

constexpr int SEL_T = 256;
constexpr int SEL_EPT = 8;                       // elements per thread in the compaction
constexpr int SEL_CHUNK = SEL_T * SEL_EPT;       // 2048 elements per block

struct SelectState {
    uint32_t prefix;      // key bits fixed so far (right-aligned)
    uint32_t pad;
    int64_t k_rem;        // how many more to take from the current bucket
};

// Workspace: [0, 3*2048*4) histograms | state | block counts (2 x int32 per block) | block offsets (2 x int64)
struct SelectWs {
    uint32_t* hist;       // [3][2048]
    SelectState* state;
    int32_t* blk_cnt;     // [nblk][2]  (gt, eq)
    int64_t* blk_off;     // [nblk][2]  exclusive prefix (gt, eq)
};

// A kernel whose gate is closed returns at once: the launches of the bracketed path and of its
// fallback are both enqueued, and a flag written on the device decides which of the two does the work.
struct Gate {
    const uint32_t* flag;     // nullptr: always open
    uint32_t want;
    __device__ __forceinline__ bool closed() const { return flag != nullptr && *flag != want; }
};

__host__ __device__ inline int64_t sel_nblk(int64_t N) { return (N + SEL_CHUNK - 1) / SEL_CHUNK; }

template <int PASS>
__global__ void __launch_bounds__(SEL_T)
select_hist_kernel(const float* __restrict__ scores, int64_t N, const SelectState* __restrict__ state,
                   uint32_t* __restrict__ hist, Gate gate)
{
    __shared__ uint32_t s_h[2048];
    if (gate.closed()) return;
    for (int i = threadIdx.x; i < 2048; i += SEL_T) s_h[i] = 0;
    __syncthreads();
    const uint32_t prefix = (PASS == 0) ? 0u : state->prefix;
    const int64_t stride = (int64_t)gridDim.x * SEL_T;
    // vector body (4 scores per load) + scalar tail
    const int64_t n4 = N >> 2;
    for (int64_t i = (int64_t)blockIdx.x * SEL_T + threadIdx.x; i < n4; i += stride) {
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(scores) + i);
        const uint32_t k[4] = {order_key(raw.x), order_key(raw.y), order_key(raw.z), order_key(raw.w)};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (PASS == 0) atomicAdd(&s_h[k[u] >> 21], 1u);
            else if (PASS == 1) { if ((k[u] >> 21) == prefix) atomicAdd(&s_h[(k[u] >> 10) & 0x7FFu], 1u); }
            else { if ((k[u] >> 10) == prefix) atomicAdd(&s_h[k[u] & 0x3FFu], 1u); }
        }
    }
    for (int64_t i = (n4 << 2) + (int64_t)blockIdx.x * SEL_T + threadIdx.x; i < N; i += stride) {
        const uint32_t k = order_key(__float_as_uint(scores[i]));
        if (PASS == 0) atomicAdd(&s_h[k >> 21], 1u);
        else if (PASS == 1) { if ((k >> 21) == prefix) atomicAdd(&s_h[(k >> 10) & 0x7FFu], 1u); }
        else { if ((k >> 10) == prefix) atomicAdd(&s_h[k & 0x3FFu], 1u); }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2048; i += SEL_T)
        if (s_h[i]) atomicAdd(&hist[i], s_h[i]);
}

// One block of 1024 threads: find the bin that holds the k_rem-th largest key, counting from the top bin
// down (block-wide prefix sum over the reversed histogram).
template <int PASS>
__global__ void __launch_bounds__(1024)
select_scan_kernel(const uint32_t* __restrict__ hist, SelectState* __restrict__ state, int64_t k, Gate gate,
                   uint32_t* __restrict__ short_flag)
{
    if (gate.closed()) return;
    constexpr int NB = (PASS == 2) ? 1024 : 2048;
    constexpr int SHIFT = (PASS == 2) ? 10 : 11;
    constexpr int PER = NB / 1024;
    __shared__ int64_t s_w[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t k_rem = (PASS == 0) ? k : state->k_rem;
    const uint32_t prefix = (PASS == 0) ? 0u : state->prefix;
    int64_t c[PER];
    int64_t mine = 0;
#pragma unroll
    for (int u = 0; u < PER; ++u) { c[u] = hist[NB - 1 - (tid * PER + u)]; mine += c[u]; }
    int64_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t a = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += a;
    }
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();            // also orders every thread's read of *state before the single write below
    int64_t pre = inc - mine;
    for (int w = 0; w < warp; ++w) pre += s_w[w];
#pragma unroll
    for (int u = 0; u < PER; ++u) {
        if (pre < k_rem && k_rem <= pre + c[u]) {       // exactly one (thread, u) satisfies this
            const int b = NB - 1 - (tid * PER + u);
            state->prefix = (prefix << SHIFT) | (uint32_t)b;
            state->k_rem = k_rem - pre;
        }
        pre += c[u];
    }
    // fewer than k_rem keys in the whole histogram: no bin was chosen; tell the caller
    if (short_flag != nullptr && tid == 1023 && pre < k_rem) *short_flag = 1u;
}

__global__ void __launch_bounds__(SEL_T)
select_count_kernel(const float* __restrict__ scores, int64_t N, int64_t nblk, const SelectState* __restrict__ state,
                    int32_t* __restrict__ blk_cnt, Gate gate)
{
    __shared__ int s_gt[SEL_T / 32], s_eq[SEL_T / 32];
    if (gate.closed()) return;
    const uint32_t T = state->prefix;
    for (int64_t blk = blockIdx.x; blk < nblk; blk += gridDim.x) {
    const int64_t base = blk * SEL_CHUNK + threadIdx.x * SEL_EPT;
    int gt = 0, eq = 0;
#pragma unroll
    for (int u = 0; u < SEL_EPT; ++u) {
        const int64_t i = base + u;
        if (i < N) {
            const uint32_t k = order_key(__float_as_uint(scores[i]));
            gt += (k > T); eq += (k == T);
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
    }
    __syncthreads();
    }
}

// Exclusive prefix sums over blocks: one block of 32 warps. Warp w scans its run of consecutive entries
// in coalesced tiles of 32 (shuffle scan, running total carried along) and writes run-local prefixes;
// after the 32 run totals are combined, a second sweep adds each run's base.
__global__ void __launch_bounds__(1024)
select_block_scan_kernel(const int32_t* __restrict__ blk_cnt, int64_t nblk, int64_t* __restrict__ blk_off, Gate gate)
{
    if (gate.closed()) return;
    __shared__ int64_t s_w[2][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t per = ((nblk + 31) / 32 + 31) / 32 * 32;          // entries per warp, a multiple of 32
    const int64_t b0 = warp * per, b1 = (b0 + per < nblk) ? b0 + per : nblk;
    const int2* cnt2 = reinterpret_cast<const int2*>(blk_cnt);
    longlong2* off2 = reinterpret_cast<longlong2*>(blk_off);
    int64_t run0 = 0, run1 = 0;
    constexpr int NB = 8;                           // tiles fetched together: one memory round trip per batch
    for (int64_t t = b0; t < b1; t += 32 * NB) {
        int2 c[NB];
#pragma unroll
        for (int q = 0; q < NB; ++q) {
            const int64_t b = t + q * 32 + lane;
            c[q] = (b < b1) ? cnt2[b] : make_int2(0, 0);
        }
#pragma unroll
        for (int q = 0; q < NB; ++q) {
            const int64_t b = t + q * 32 + lane;
            int i0 = c[q].x, i1 = c[q].y;           // a tile sums to at most 32 * 4096
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int a0 = __shfl_up_sync(0xFFFFFFFFu, i0, o), a1 = __shfl_up_sync(0xFFFFFFFFu, i1, o);
                if (lane >= o) { i0 += a0; i1 += a1; }
            }
            if (b < b1) off2[b] = make_longlong2(run0 + (i0 - c[q].x), run1 + (i1 - c[q].y));
            run0 += __shfl_sync(0xFFFFFFFFu, i0, 31);
            run1 += __shfl_sync(0xFFFFFFFFu, i1, 31);
        }
    }
    if (lane == 0) { s_w[0][warp] = run0; s_w[1][warp] = run1; }
    __syncthreads();
    if (warp == 0) return;
    int64_t base0 = 0, base1 = 0;
    for (int w = 0; w < warp; ++w) { base0 += s_w[0][w]; base1 += s_w[1][w]; }
    for (int64_t t = b0; t < b1; t += 32 * NB) {
        longlong2 v[NB];
#pragma unroll
        for (int q = 0; q < NB; ++q) {
            const int64_t b = t + q * 32 + lane;
            if (b < b1) v[q] = off2[b];             // this lane's own writes of the first sweep
        }
#pragma unroll
        for (int q = 0; q < NB; ++q) {
            const int64_t b = t + q * 32 + lane;
            if (b < b1) { v[q].x += base0; v[q].y += base1; off2[b] = v[q]; }
        }
    }
}

// The same prefix sums for many blocks, spread over the GPU (one SM alone is bound by its own memory
// bandwidth): tiles of 1024 entries are scanned by a block each, which also leaves the tile's total;
// a second launch adds to every tile the sum of the totals of the tiles before it.
__global__ void __launch_bounds__(1024)
select_tile_scan_kernel(const int32_t* __restrict__ blk_cnt, int64_t nblk, int64_t* __restrict__ blk_off,
                        int64_t* __restrict__ tile_tot, Gate gate)
{
    if (gate.closed()) return;
    __shared__ int s_w[2][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t b = (int64_t)blockIdx.x * 1024 + threadIdx.x;
    int2 c = make_int2(0, 0);
    if (b < nblk) c = reinterpret_cast<const int2*>(blk_cnt)[b];
    int i0 = c.x, i1 = c.y;                         // a tile sums to at most 1024 * 4096
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a0 = __shfl_up_sync(0xFFFFFFFFu, i0, o), a1 = __shfl_up_sync(0xFFFFFFFFu, i1, o);
        if (lane >= o) { i0 += a0; i1 += a1; }
    }
    if (lane == 31) { s_w[0][warp] = i0; s_w[1][warp] = i1; }
    __syncthreads();
    const int w0 = s_w[0][lane], w1 = s_w[1][lane];
    int p0 = w0, p1 = w1;                           // every warp scans the 32 warp totals
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a0 = __shfl_up_sync(0xFFFFFFFFu, p0, o), a1 = __shfl_up_sync(0xFFFFFFFFu, p1, o);
        if (lane >= o) { p0 += a0; p1 += a1; }
    }
    const int base0 = __shfl_sync(0xFFFFFFFFu, p0 - w0, warp), base1 = __shfl_sync(0xFFFFFFFFu, p1 - w1, warp);
    if (b < nblk) reinterpret_cast<longlong2*>(blk_off)[b] = make_longlong2((int64_t)(base0 + i0 - c.x), (int64_t)(base1 + i1 - c.y));
    if (threadIdx.x == 1023)
        reinterpret_cast<longlong2*>(tile_tot)[blockIdx.x] = make_longlong2((int64_t)(base0 + i0), (int64_t)(base1 + i1));
}

__global__ void __launch_bounds__(1024)
select_tile_add_kernel(int64_t nblk, int64_t* __restrict__ blk_off, const int64_t* __restrict__ tile_tot, Gate gate)
{
    if (gate.closed()) return;
    if (blockIdx.x == 0) return;
    __shared__ int64_t s_w[2][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t a0 = 0, a1 = 0;
    for (int64_t t = threadIdx.x; t < (int64_t)blockIdx.x; t += 1024) {
        const longlong2 v = reinterpret_cast<const longlong2*>(tile_tot)[t];
        a0 += v.x; a1 += v.y;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { a0 += __shfl_xor_sync(0xFFFFFFFFu, a0, o); a1 += __shfl_xor_sync(0xFFFFFFFFu, a1, o); }
    if (lane == 0) { s_w[0][warp] = a0; s_w[1][warp] = a1; }
    __syncthreads();
    int64_t base0 = 0, base1 = 0;
#pragma unroll
    for (int w = 0; w < 32; ++w) { base0 += s_w[0][w]; base1 += s_w[1][w]; }
    const int64_t b = (int64_t)blockIdx.x * 1024 + threadIdx.x;
    if (b < nblk) {
        longlong2 v = reinterpret_cast<longlong2*>(blk_off)[b];
        v.x += base0; v.y += base1;
        reinterpret_cast<longlong2*>(blk_off)[b] = v;
    }
}

// Prefix sums over the per-block counts: one launch for a few thousand blocks, two beyond.
inline void launch_block_scan(const int32_t* blk_cnt, int64_t nblk, int64_t* blk_off, int64_t* tile_tot, Gate gate,
                              cudaStream_t st)
{
    if (tile_tot == nullptr || nblk <= 4096) {
        select_block_scan_kernel<<<1, 1024, 0, st>>>(blk_cnt, nblk, blk_off, gate);
        count_launches(1);
    } else {
        const unsigned tiles = (unsigned)((nblk + 1023) / 1024);
        select_tile_scan_kernel<<<tiles, 1024, 0, st>>>(blk_cnt, nblk, blk_off, tile_tot, gate);
        select_tile_add_kernel<<<tiles, 1024, 0, st>>>(nblk, blk_off, tile_tot, gate);
        count_launches(2);
    }
}

__global__ void __launch_bounds__(SEL_T)
select_write_kernel(const float* __restrict__ scores, int64_t N, int64_t nblk, const SelectState* __restrict__ state,
                    const int64_t* __restrict__ blk_off, int64_t* __restrict__ indices, Gate gate)
{
    __shared__ int s_gt[SEL_T / 32], s_eq[SEL_T / 32];
    if (gate.closed()) return;
    const uint32_t T = state->prefix;
    const int64_t k_ties = state->k_rem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t blk = blockIdx.x; blk < nblk; blk += gridDim.x) {
    const int64_t base = blk * SEL_CHUNK + threadIdx.x * SEL_EPT;
    uint32_t fgt = 0, feq = 0;
#pragma unroll
    for (int u = 0; u < SEL_EPT; ++u) {
        const int64_t i = base + u;
        if (i < N) {
            const uint32_t k = order_key(__float_as_uint(scores[i]));
            fgt |= (uint32_t)(k > T) << u; feq |= (uint32_t)(k == T) << u;
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
    int64_t gt_before = blk_off[2 * blk] + igt - gt;
    int64_t eq_before = blk_off[2 * blk + 1] + ieq - eq;
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
    __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// Large N: two reads of the scores instead of five. A stratified sample brackets the k-th largest
// key from below (lo); one pass over the scores copies every key >= lo, in index order, into the
// segment of its 4096-score chunk; the radix select and the ordered compaction then run on those
// candidates alone (a few per cent of N, resident in L2). If fewer than k candidates turn up (the
// bracket was too high: probability below 1e-8 for scores in any order, since the offset inside
// each stratum is hashed) a flag opens the gates of the exact multi-pass path enqueued behind.
// ------------------------------------------------------------------------------------------------

constexpr int SG_T = 256;
constexpr int SG_CH = 4096;                     // scores per chunk = capacity of its candidate segment
constexpr int SG_SAMPLE = 16384;                // strata (one sampled score each)
constexpr int64_t SG_MIN_N = (int64_t)1 << 22;  // above this the bracketed path is used

struct BracketState {
    uint32_t lo_key;              // candidates are the keys >= lo_key
    uint32_t fallback;            // 1: fewer than k candidates, the exact path must run
    unsigned long long n_cand;
};

struct BracketWs {
    uint32_t* hist;               // [6][2048]: 0..2 candidates, 3..5 fallback
    SelectState* state;           // 256-byte region; BracketState sits 64 bytes in
    BracketState* bstate;
    int64_t* blk_off;             // sized for the fallback's 2048-score blocks
    int32_t* blk_cnt;
    int64_t* tile_tot;            // [ceil(nblk / 1024)][2] totals of the block-count tiles
    uint32_t* sample_key;         // [SG_SAMPLE]
    uint32_t* chunk_cnt;          // [nchunk]
    uint16_t* seg_off;            // [nchunk][SG_CH] offset of the candidate inside its chunk
    uint32_t* seg_key;            // [nchunk][SG_CH]
};

__host__ __device__ inline int64_t sg_nchunk(int64_t N) { return (N + SG_CH - 1) / SG_CH; }

__device__ __forceinline__ uint32_t mix32(uint32_t x)
{
    x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
    return x;
}

// First launch of the bracketed path, spread over the GPU: clears the histograms and the state, and
// fetches one score per stratum (16384 scattered reads: far too many misses for one SM to keep in flight).
__global__ void __launch_bounds__(256)
select_init_kernel(const float* __restrict__ scores, int64_t N, uint32_t* __restrict__ clear, int clear_words,
                   uint32_t* __restrict__ sample_key)
{
    const int j = blockIdx.x * 256 + threadIdx.x;           // grid covers SG_SAMPLE threads
    for (int i = j; i < clear_words; i += SG_SAMPLE) clear[i] = 0u;
    const int64_t per = N / SG_SAMPLE;                      // >= 256 for every N this path takes
    // offset inside the stratum: hash scaled to [0, per) (per < 2^32 for every N below 2^46)
    const int64_t pos = (int64_t)j * per + (int64_t)(((uint64_t)mix32(0x9E3779B9u * (uint32_t)j + 0x85EBCA6Bu) * (uint64_t)per) >> 32);
    sample_key[j] = order_key(__float_as_uint(__ldg(scores + pos)));
}

// One block: the r-th largest sampled key by bisection on the key's bits, largest t with
// #{key >= t} >= r: 32 block-wide counts over 16 keys per thread held in registers.
// r = expected rank of the k-th largest + 6 standard deviations + 8.
__global__ void __launch_bounds__(1024)
select_sample_kernel(const uint32_t* __restrict__ sample_key, int64_t N, int64_t k, BracketState* __restrict__ bs,
                     int force_short)
{
    constexpr int PER_T = SG_SAMPLE / 1024;
    __shared__ int s_cnt[2][32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const double p = (double)k / (double)N;
    const double ks = ceil(p * (double)SG_SAMPLE);
    const double rr = ks + ceil(6.0 * sqrt(ks * (1.0 - p))) + 8.0;
    if (force_short) { if (tid == 0) bs->lo_key = 0xFF800000u; return; }      // key of +inf
    if (rr >= (double)SG_SAMPLE) { if (tid == 0) bs->lo_key = 0u; return; }     // every score is a candidate
    const int r = (int)rr;
    uint32_t v[PER_T];
#pragma unroll
    for (int i = 0; i < PER_T; ++i) v[i] = sample_key[tid + i * 1024];
    uint32_t t = 0;
#pragma unroll 1
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t cand = t | (1u << bit);
        int c = 0;
#pragma unroll
        for (int i = 0; i < PER_T; ++i) c += (v[i] >= cand);
        c = __reduce_add_sync(0xFFFFFFFFu, c);
        if (lane == 0) s_cnt[bit & 1][warp] = c;
        __syncthreads();                    // the two count buffers alternate: one barrier per bit
        const int total = __reduce_add_sync(0xFFFFFFFFu, s_cnt[bit & 1][lane]);
        if (total >= r) t = cand;
    }
    if (tid == 0) bs->lo_key = t;
}

// The second (and last) read of the scores: the candidates of each 4096-score chunk go to the chunk's
// segment (key and offset inside the chunk, in no particular order: the final write restores index
// order from the offsets), and their top-11-bit histogram feeds the first round of the radix select.
// The test runs on s = key ^ 0x80000000 read as a signed integer: lo_s <= s <= s(+inf), one subtraction
// and one unsigned compare. For a bracket above zero (POS) s is the raw bit pattern itself: negative
// scores and NaNs fall outside the range by themselves. Otherwise s takes two more operations per score.
// A warp owns whole chunks and walks each in eight steps of 512 scores (16 per lane, as four 16-byte
// pieces 128 scores apart), with no block-wide barrier; a warp scan of the per-lane counts gives each
// lane its run in the segment. Each lane fetches its own pieces with cp.async into a ring of three
// steps, two steps ahead of the one it works on: enough bytes in flight per SM without registers.
constexpr int SG_RING = 3;
constexpr int SG_STEP = 512;                    // scores per warp step
constexpr int SG_STEPS = SG_CH / SG_STEP;       // 8

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int KEEP> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(KEEP) : "memory"); }

template <bool POS>
__device__ __forceinline__ void gather_chunks(const float* __restrict__ scores, int64_t N, uint32_t lo,
                                              uint32_t* __restrict__ seg_key, uint16_t* __restrict__ seg_off,
                                              uint32_t* __restrict__ chunk_cnt, uint32_t* s_h, uint32_t* __restrict__ hist0,
                                              uint32_t* s_ring /* this warp's [SG_RING][SG_STEP] */, unsigned long long& mine)
{
    const int lane = threadIdx.x & 31;
    const uint32_t lo_s = lo ^ 0x80000000u;
    const uint32_t range = (lo == 0u) ? 0xFFFFFFFFu : (0x7F800000u - lo_s);     // lo == 0: NaNs are candidates too
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
        uint32_t* kp = seg_key + c * SG_CH;
        uint16_t* op = seg_off + c * SG_CH;
        uint32_t run = 0;
#pragma unroll 1
        for (int sub = 0; sub < SG_STEPS; ++sub) {
            fetch();
            cp_async_wait<2>();                                       // this lane's pieces of the step have landed
            const uint32_t* mine_s = s_ring + slot * SG_STEP + lane * 4;
            const int64_t i0 = c * SG_CH + sub * SG_STEP;
            uint32_t F = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint4 raw = *reinterpret_cast<const uint4*>(mine_s + j * 128);
                const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t sv = POS ? r[u] : (r[u] ^ ((uint32_t)((int32_t)r[u] >> 31) & 0x7FFFFFFFu));
                    if (sv - lo_s <= range) F |= 1u << (4 * j + u);
                }
            }
            if (N - i0 < SG_STEP) {                                   // ragged end: drop what lies beyond N
                uint32_t valid = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t left = N - (i0 + lane * 4 + j * 128);
                    valid |= (left >= 4 ? 0xFu : (left > 0 ? (1u << (int)left) - 1u : 0u)) << (4 * j);
                }
                F &= valid;
            }
            const uint32_t cnt = (uint32_t)__popc(F);
            uint32_t inc = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t a = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                if (lane >= o) inc += a;
            }
            const uint32_t tot = __shfl_sync(0xFFFFFFFFu, inc, 31);
            uint32_t pos = run + inc - cnt;
            const uint32_t obase = (uint32_t)(sub * SG_STEP + lane * 4);
            while (F) {
                const int b = __ffs((int)F) - 1;
                F &= F - 1u;
                const uint32_t e = (uint32_t)((b >> 2) * 128 + (b & 3));
                const uint32_t r = mine_s[e];
                // the key; a NaN (only reachable with lo == 0) has key 0
                const uint32_t key = POS ? (r | 0x80000000u) : order_key(r);
                kp[pos] = key;
                op[pos] = (uint16_t)(obase + e);
                if (POS || key >= 0x80000000u) atomicAdd(&s_h[(key >> 21) - 1024u], 1u);
                else atomicAdd(&hist0[key >> 21], 1u);          // negative scores and NaNs: rare as candidates
                ++pos;
            }
            run += tot;
            slot = (slot == SG_RING - 1) ? 0 : slot + 1;
        }
        if (lane == 0) { chunk_cnt[c] = run; mine += run; }
    }
    cp_async_wait<0>();
}

__global__ void __launch_bounds__(SG_T, 4)
select_gather_kernel(const float* __restrict__ scores, int64_t N, BracketState* __restrict__ bs,
                     uint32_t* __restrict__ seg_key, uint16_t* __restrict__ seg_off,
                     uint32_t* __restrict__ chunk_cnt, uint32_t* __restrict__ hist0)
{
    extern __shared__ __align__(16) uint8_t s_dyn[];      // per warp: ring of SG_RING steps of raw scores
    __shared__ uint32_t s_h[1024];           // bins 1024..2047: keys of scores with the sign bit clear
    const int tid = threadIdx.x;
    for (int i = tid; i < 1024; i += SG_T) s_h[i] = 0;
    __syncthreads();
    const uint32_t lo = bs->lo_key;
    unsigned long long mine = 0;
    uint32_t* s_ring = reinterpret_cast<uint32_t*>(s_dyn) + (tid >> 5) * (SG_RING * SG_STEP);
    if (lo > 0x80000000u) gather_chunks<true>(scores, N, lo, seg_key, seg_off, chunk_cnt, s_h, hist0, s_ring, mine);
    else gather_chunks<false>(scores, N, lo, seg_key, seg_off, chunk_cnt, s_h, hist0, s_ring, mine);
    __syncthreads();
    for (int i = tid; i < 1024; i += SG_T)
        if (s_h[i]) atomicAdd(&hist0[1024 + i], s_h[i]);
    if ((tid & 31) == 0 && mine) atomicAdd(&bs->n_cand, mine);
}

// The kernels below walk the candidate segments with one warp per chunk. A segment holds a few hundred
// entries, so the walk is bound by memory round trips, not bytes: each warp fetches the first CB * 32
// keys of its NEXT chunk (and the count of the one after) before it works on the current one.
constexpr int CB = 8;

struct SegCursor {
    const uint32_t* __restrict__ seg_key;
    const uint32_t* __restrict__ chunk_cnt;
    int64_t nchunk, nwarp, c;
    int lane;
    int cnt, cnt_next;                  // of chunk c and of chunk c + nwarp
    uint32_t k[CB], k_next[CB];         // first batch of chunk c / c + nwarp (lanes beyond the count: unspecified)

    __device__ __forceinline__ void fetch_keys(int64_t chunk, int n, uint32_t (&dst)[CB]) const
    {
        const uint32_t* seg = seg_key + chunk * SG_CH;
#pragma unroll
        for (int q = 0; q < CB; ++q) {
            const int j = q * 32 + lane;
            if (j < n) dst[q] = __ldg(seg + j);
        }
    }
    __device__ __forceinline__ void start(const uint32_t* sk, const uint32_t* cc, int64_t n)
    {
        seg_key = sk; chunk_cnt = cc; nchunk = n;
        lane = threadIdx.x & 31;
        nwarp = (int64_t)gridDim.x * (blockDim.x >> 5);
        c = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
        cnt = (c < nchunk) ? (int)__ldg(chunk_cnt + c) : 0;
        cnt_next = (c + nwarp < nchunk) ? (int)__ldg(chunk_cnt + c + nwarp) : 0;
        if (c < nchunk) fetch_keys(c, cnt, k);
    }
    __device__ __forceinline__ bool valid() const { return c < nchunk; }
    // issue the loads for the chunks ahead; call before working on chunk c
    __device__ __forceinline__ int prefetch()
    {
        const int cnt_after = (c + 2 * nwarp < nchunk) ? (int)__ldg(chunk_cnt + c + 2 * nwarp) : 0;
        if (c + nwarp < nchunk) fetch_keys(c + nwarp, cnt_next, k_next);
        return cnt_after;
    }
    __device__ __forceinline__ void advance(int cnt_after)
    {
        c += nwarp; cnt = cnt_next; cnt_next = cnt_after;
#pragma unroll
        for (int q = 0; q < CB; ++q) k[q] = k_next[q];
    }
};

// Radix-select rounds 2 and 3 on the candidates.
template <int PASS>
__global__ void __launch_bounds__(SG_T)
cand_hist_kernel(const uint32_t* __restrict__ seg_key, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk,
                 const SelectState* __restrict__ state, uint32_t* __restrict__ hist, Gate gate)
{
    __shared__ uint32_t s_h[2048];
    if (gate.closed()) return;
    for (int i = threadIdx.x; i < 2048; i += blockDim.x) s_h[i] = 0;
    __syncthreads();
    const uint32_t prefix = state->prefix;
    auto add = [&](uint32_t key) {
        if (PASS == 1) { if ((key >> 21) == prefix) atomicAdd(&s_h[(key >> 10) & 0x7FFu], 1u); }
        else { if ((key >> 10) == prefix) atomicAdd(&s_h[key & 0x3FFu], 1u); }
    };
    SegCursor cur;
    for (cur.start(seg_key, chunk_cnt, nchunk); cur.valid();) {
        const int after = cur.prefetch();
#pragma unroll
        for (int q = 0; q < CB; ++q)
            if (q * 32 + cur.lane < cur.cnt) add(cur.k[q]);
        const uint32_t* seg = seg_key + cur.c * SG_CH;
        for (int j = CB * 32 + cur.lane; j < cur.cnt; j += 32) add(seg[j]);       // segments longer than a batch
        cur.advance(after);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2048; i += blockDim.x)
        if (s_h[i]) atomicAdd(&hist[i], s_h[i]);
}

__global__ void __launch_bounds__(SG_T)
cand_count_kernel(const uint32_t* __restrict__ seg_key, const uint32_t* __restrict__ chunk_cnt, int64_t nchunk,
                  const SelectState* __restrict__ state, int32_t* __restrict__ blk_cnt, Gate gate)
{
    if (gate.closed()) return;
    const uint32_t T = state->prefix;
    SegCursor cur;
    for (cur.start(seg_key, chunk_cnt, nchunk); cur.valid();) {
        const int after = cur.prefetch();
        int gt = 0, eq = 0;
#pragma unroll
        for (int q = 0; q < CB; ++q)
            if (q * 32 + cur.lane < cur.cnt) { gt += (cur.k[q] > T); eq += (cur.k[q] == T); }
        const uint32_t* seg = seg_key + cur.c * SG_CH;
        for (int j = CB * 32 + cur.lane; j < cur.cnt; j += 32) { const uint32_t key = seg[j]; gt += (key > T); eq += (key == T); }
        gt = __reduce_add_sync(0xFFFFFFFFu, gt);
        eq = __reduce_add_sync(0xFFFFFFFFu, eq);
        if (cur.lane == 0) *reinterpret_cast<int2*>(blk_cnt + 2 * cur.c) = make_int2(gt, eq);
        cur.advance(after);
    }
}

// Final write: a warp per chunk marks the offsets of {key > T} and of {key == T} in two 4096-bit maps
// in shared memory, which puts the segment's unordered candidates back in index order: the number of
// set bits below a candidate's offset (a per-word prefix plus a masked population count) is how many
// of the chunk's larger or equal-key scores come before it, and with the chunk's offsets that is its
// place in the output.
__global__ void __launch_bounds__(SG_T)
cand_write_kernel(const uint32_t* __restrict__ seg_key, const uint16_t* __restrict__ seg_off,
                  const uint32_t* __restrict__ chunk_cnt, int64_t nchunk, const SelectState* __restrict__ state,
                  const int64_t* __restrict__ blk_off, int64_t* __restrict__ indices, Gate gate)
{
    __shared__ __align__(16) uint32_t s_bm[SG_T / 32][2][SG_CH / 32];
    __shared__ __align__(16) uint16_t s_pre[SG_T / 32][2][SG_CH / 32];      // set bits in the words before
    if (gate.closed()) return;
    const uint32_t T = state->prefix;
    const int64_t k_ties = state->k_rem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* bm_gt = s_bm[warp][0];
    uint32_t* bm_eq = s_bm[warp][1];
    uint16_t* pre_gt = s_pre[warp][0];
    uint16_t* pre_eq = s_pre[warp][1];
    SegCursor cur;
    for (cur.start(seg_key, chunk_cnt, nchunk); cur.valid();) {
        const int after = cur.prefetch();
        const int64_t c = cur.c;
        const int cnt = cur.cnt;
        if (cnt == 0) { cur.advance(after); continue; }
        const uint32_t* seg = seg_key + c * SG_CH;
        const uint16_t* off = seg_off + c * SG_CH;
        const longlong2 base2 = *reinterpret_cast<const longlong2*>(blk_off + 2 * c);
        // offsets of the first batch, for the entries that are selected or tied (all loads issued together)
        uint32_t o[CB];
#pragma unroll
        for (int q = 0; q < CB; ++q) {
            const int j = q * 32 + lane;
            o[q] = (j < cnt && cur.k[q] >= T) ? (uint32_t)off[j] : 0xFFFFFFFFu;
        }
        reinterpret_cast<uint4*>(bm_gt)[lane] = make_uint4(0u, 0u, 0u, 0u);
        reinterpret_cast<uint4*>(bm_eq)[lane] = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
#pragma unroll
        for (int q = 0; q < CB; ++q)
            if (o[q] != 0xFFFFFFFFu) atomicOr((cur.k[q] > T ? bm_gt : bm_eq) + (o[q] >> 5), 1u << (o[q] & 31u));
        for (int j = CB * 32 + lane; j < cnt; j += 32) {                 // segments longer than a batch
            const uint32_t key = seg[j];
            if (key >= T) { const uint32_t oo = off[j]; atomicOr((key > T ? bm_gt : bm_eq) + (oo >> 5), 1u << (oo & 31u)); }
        }
        __syncwarp();
        const uint4 g4 = reinterpret_cast<const uint4*>(bm_gt)[lane];
        const uint4 e4 = reinterpret_cast<const uint4*>(bm_eq)[lane];
        const int pg[4] = {__popc(g4.x), __popc(g4.y), __popc(g4.z), __popc(g4.w)};
        const int pe[4] = {__popc(e4.x), __popc(e4.y), __popc(e4.z), __popc(e4.w)};
        const int cg = pg[0] + pg[1] + pg[2] + pg[3], ce = pe[0] + pe[1] + pe[2] + pe[3];
        int ig = cg, ie = ce;
#pragma unroll
        for (int sh = 1; sh < 32; sh <<= 1) {
            const int a2 = __shfl_up_sync(0xFFFFFFFFu, ig, sh), b2 = __shfl_up_sync(0xFFFFFFFFu, ie, sh);
            if (lane >= sh) { ig += a2; ie += b2; }
        }
        ig -= cg; ie -= ce;
        reinterpret_cast<uint2*>(pre_gt)[lane] = make_uint2((uint32_t)ig | ((uint32_t)(ig + pg[0]) << 16),
                                                            (uint32_t)(ig + pg[0] + pg[1]) | ((uint32_t)(ig + pg[0] + pg[1] + pg[2]) << 16));
        reinterpret_cast<uint2*>(pre_eq)[lane] = make_uint2((uint32_t)ie | ((uint32_t)(ie + pe[0]) << 16),
                                                            (uint32_t)(ie + pe[0] + pe[1]) | ((uint32_t)(ie + pe[0] + pe[1] + pe[2]) << 16));
        __syncwarp();
        // place = (larger keys before) + min(ties before, k_ties): the chunk's own part of both in 32 bits
        const int64_t room64 = k_ties - base2.y;                                  // ties this chunk may still admit
        const uint32_t room = room64 <= 0 ? 0u : (room64 >= SG_CH ? (uint32_t)SG_CH : (uint32_t)room64);
        int64_t* out = indices + base2.x + (base2.y < k_ties ? base2.y : k_ties);
        const int64_t ibase = c * SG_CH;
        auto place = [&](uint32_t key, uint32_t oo) {
            const uint32_t w = oo >> 5, below = (1u << (oo & 31u)) - 1u;
            const uint32_t g_loc = pre_gt[w] + __popc(bm_gt[w] & below);
            const uint32_t e_loc = pre_eq[w] + __popc(bm_eq[w] & below);
            if (key > T || e_loc < room) out[g_loc + (e_loc < room ? e_loc : room)] = ibase + oo;
        };
#pragma unroll
        for (int q = 0; q < CB; ++q)
            if (o[q] != 0xFFFFFFFFu) place(cur.k[q], o[q]);
        for (int j = CB * 32 + lane; j < cnt; j += 32) {
            const uint32_t key = seg[j];
            if (key >= T) place(key, off[j]);
        }
        __syncwarp();       // the maps are cleared again for the warp's next chunk
        cur.advance(after);
    }
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
    const int64_t nblk = sel_nblk(N);
    w.blk_off = reinterpret_cast<int64_t*>(p); p += align_up((size_t)nblk * 2 * sizeof(int64_t), 256);
    w.blk_cnt = reinterpret_cast<int32_t*>(p);
    return w;
}

size_t compact_workspace_bytes(int64_t N)
{
    const int64_t nblk = sel_nblk(N > 0 ? N : 1);
    return 3 * 2048 * sizeof(uint32_t) + 256 + align_up((size_t)nblk * 2 * sizeof(int64_t), 256) +
           align_up((size_t)nblk * 2 * sizeof(int32_t), 256);
}

BracketWs carve_bracket(void* ws, int64_t N)
{
    BracketWs w;
    uint8_t* p = reinterpret_cast<uint8_t*>(ws);
    w.hist = reinterpret_cast<uint32_t*>(p); p += 6 * 2048 * sizeof(uint32_t);
    w.state = reinterpret_cast<SelectState*>(p);
    w.bstate = reinterpret_cast<BracketState*>(p + 64); p += 256;
    const int64_t nblk = sel_nblk(N), nchunk = sg_nchunk(N);
    w.blk_off = reinterpret_cast<int64_t*>(p); p += align_up((size_t)nblk * 2 * sizeof(int64_t), 256);
    w.blk_cnt = reinterpret_cast<int32_t*>(p); p += align_up((size_t)nblk * 2 * sizeof(int32_t), 256);
    w.tile_tot = reinterpret_cast<int64_t*>(p); p += align_up((size_t)((nblk + 1023) / 1024) * 2 * sizeof(int64_t), 256);
    w.sample_key = reinterpret_cast<uint32_t*>(p); p += SG_SAMPLE * sizeof(uint32_t);
    w.chunk_cnt = reinterpret_cast<uint32_t*>(p); p += align_up((size_t)nchunk * sizeof(uint32_t), 256);
    w.seg_off = reinterpret_cast<uint16_t*>(p); p += align_up((size_t)nchunk * SG_CH * sizeof(uint16_t), 256);
    w.seg_key = reinterpret_cast<uint32_t*>(p);
    return w;
}

size_t bracket_workspace_bytes(int64_t N)
{
    const int64_t nblk = sel_nblk(N), nchunk = sg_nchunk(N);
    return 6 * 2048 * sizeof(uint32_t) + 256 + align_up((size_t)nblk * 2 * sizeof(int64_t), 256) +
           align_up((size_t)nblk * 2 * sizeof(int32_t), 256) + align_up((size_t)((nblk + 1023) / 1024) * 2 * sizeof(int64_t), 256) +
           SG_SAMPLE * sizeof(uint32_t) + align_up((size_t)nchunk * sizeof(uint32_t), 256) +
           align_up((size_t)nchunk * SG_CH * sizeof(uint16_t), 256) + (size_t)nchunk * SG_CH * sizeof(uint32_t);
}

// The exact multi-pass path on the scores themselves (five reads). hist: three cleared histograms.
cudaError_t launch_multipass(const float* scores, int64_t N, int64_t k, int64_t* indices, uint32_t* hist,
                             SelectState* state, int32_t* blk_cnt, int64_t* blk_off, int64_t* tile_tot, Gate gate, cudaStream_t st)
{
    int64_t hb = (N / 4 + SEL_T - 1) / SEL_T;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (hb > cap) hb = cap;
    if (hb < 1) hb = 1;
    select_hist_kernel<0><<<(unsigned)hb, SEL_T, 0, st>>>(scores, N, state, hist, gate);
    select_scan_kernel<0><<<1, 1024, 0, st>>>(hist, state, k, gate, nullptr);
    select_hist_kernel<1><<<(unsigned)hb, SEL_T, 0, st>>>(scores, N, state, hist + 2048, gate);
    select_scan_kernel<1><<<1, 1024, 0, st>>>(hist + 2048, state, k, gate, nullptr);
    select_hist_kernel<2><<<(unsigned)hb, SEL_T, 0, st>>>(scores, N, state, hist + 4096, gate);
    select_scan_kernel<2><<<1, 1024, 0, st>>>(hist + 4096, state, k, gate, nullptr);
    const int64_t nblk = sel_nblk(N);
    const int64_t cap2 = (int64_t)sm_count() * 32;
    const unsigned cg = (unsigned)(nblk < cap2 ? nblk : cap2);
    select_count_kernel<<<cg, SEL_T, 0, st>>>(scores, N, nblk, state, blk_cnt, gate);
    launch_block_scan(blk_cnt, nblk, blk_off, tile_tot, gate, st);
    select_write_kernel<<<cg, SEL_T, 0, st>>>(scores, N, nblk, state, blk_off, indices, gate);
    count_launches(8);
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
    cudaError_t e = cudaSuccess;
    const int64_t nchunk = sg_nchunk(N);
    const int64_t cap = (int64_t)sm_count() * 8;
    const int64_t gcap = (int64_t)sm_count() * 4;          // the gather kernel's resident blocks (48 KiB ring each)
    const int64_t gneed = (nchunk + SG_T / 32 - 1) / (SG_T / 32);       // a warp per chunk
    const unsigned gb = (unsigned)(gneed < gcap ? gneed : gcap);
    const int64_t wb = (nchunk + SG_T / 32 - 1) / (SG_T / 32);
    const unsigned cb = (unsigned)(wb < cap ? wb : cap);
    const Gate none{nullptr, 0u};
    const Gate ok{&w.bstate->fallback, 0u};          // enough candidates: select among them
    const Gate fb{&w.bstate->fallback, 1u};          // too few: exact path on the scores
    select_init_kernel<<<SG_SAMPLE / 256, 256, 0, st>>>(scores, N, w.hist, 6 * 2048 + 64, w.sample_key);     // histograms + state
    select_sample_kernel<<<1, 1024, 0, st>>>(w.sample_key, N, k, w.bstate, force_short ? 1 : 0);
    select_gather_kernel<<<gb, SG_T, (SG_T / 32) * SG_RING * SG_STEP * sizeof(uint32_t), st>>>(scores, N, w.bstate, w.seg_key, w.seg_off, w.chunk_cnt, w.hist);
    select_scan_kernel<0><<<1, 1024, 0, st>>>(w.hist, w.state, k, none, &w.bstate->fallback);
    cand_hist_kernel<1><<<cb, SG_T, 0, st>>>(w.seg_key, w.chunk_cnt, nchunk, w.state, w.hist + 2048, ok);
    select_scan_kernel<1><<<1, 1024, 0, st>>>(w.hist + 2048, w.state, k, ok, nullptr);
    cand_hist_kernel<2><<<cb, SG_T, 0, st>>>(w.seg_key, w.chunk_cnt, nchunk, w.state, w.hist + 4096, ok);
    select_scan_kernel<2><<<1, 1024, 0, st>>>(w.hist + 4096, w.state, k, ok, nullptr);
    cand_count_kernel<<<cb, SG_T, 0, st>>>(w.seg_key, w.chunk_cnt, nchunk, w.state, w.blk_cnt, ok);
    launch_block_scan(w.blk_cnt, nchunk, w.blk_off, w.tile_tot, ok, st);
    cand_write_kernel<<<cb, SG_T, 0, st>>>(w.seg_key, w.seg_off, w.chunk_cnt, nchunk, w.state, w.blk_off, indices, ok);
    count_launches(10);          // the prefix-sum launches count themselves
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_multipass(scores, N, k, indices, w.hist + 3 * 2048, w.state, w.blk_cnt, w.blk_off, w.tile_tot, fb, st);
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
    cudaError_t e = cudaMemsetAsync(w.hist, 0, 3 * 2048 * sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    return launch_multipass(scores, N, k, indices, w.hist, w.state, w.blk_cnt, w.blk_off, nullptr, Gate{nullptr, 0u}, st);
}

}  // namespace qless

// ------------------------------------------------------------------------------------------------
// Selection without any allocation: the scratch of the radix select lives in a fixed device array.
// ------------------------------------------------------------------------------------------------

namespace qless {
namespace {

// 3 histograms (24 KiB) + state (256 B) + per-block offsets and counts for MAX_N / 2048 = 2048 blocks
// (32 KiB + 16 KiB) = 73 984 bytes; rounded up. Resident on every GPU that loads the library.
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
        static_assert(kStaticScratchBytes >= 3 * 2048 * 4 + 256 + 2048 * 16 + 2048 * 8, "scratch array too small");
        QLESS_REQUIRE(select_workspace_bytes(N) <= kStaticScratchBytes, QLESS_ERR_UNSUPPORTED, "internal: scratch array too small");
    }
    *k_out = k;
    if (k == 0) return QLESS_OK;
    void* scratch = nullptr;
    qless_status s = static_scratch(&scratch);
    if (s != QLESS_OK) return s;
    // The histograms are cleared inside; the state and the per-block arrays are rewritten in full for
    // this N before they are read, so nothing of the previous call's contents is used.
    QLESS_CUDA_TRY(launch_select_topk(scores, N, k, indices, scratch, st));
    return QLESS_OK;
}
