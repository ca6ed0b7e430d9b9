// Stage 4: top-k by radix select on order-preserving 32-bit keys, then an index-ordered compaction.
// Three histogram passes (11 + 11 + 10 bits) fix the k-th largest key T exactly and the number of
// keys equal to T that are admitted (smallest indices first); the compaction writes the indices of
// {key > T} and of the admitted ties in ascending order.
#include <cmath>
#include <mutex>

#include "qless_kernels.h"

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

__host__ __device__ inline int64_t sel_nblk(int64_t N) { return (N + SEL_CHUNK - 1) / SEL_CHUNK; }

template <int PASS>
__global__ void __launch_bounds__(SEL_T)
select_hist_kernel(const float* __restrict__ scores, int64_t N, const SelectState* __restrict__ state,
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
select_scan_kernel(const uint32_t* __restrict__ hist, SelectState* __restrict__ state, int64_t k)
{
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
}

__global__ void __launch_bounds__(SEL_T)
select_count_kernel(const float* __restrict__ scores, int64_t N, const SelectState* __restrict__ state,
                    int32_t* __restrict__ blk_cnt)
{
    __shared__ int s_gt[SEL_T / 32], s_eq[SEL_T / 32];
    const uint32_t T = state->prefix;
    const int64_t base = (int64_t)blockIdx.x * SEL_CHUNK + threadIdx.x * SEL_EPT;
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
        blk_cnt[2 * blockIdx.x] = a; blk_cnt[2 * blockIdx.x + 1] = b;
    }
}

// Exclusive prefix sums over blocks (one block of 1024 threads, sequential over tiles of 1024 blocks).
__global__ void __launch_bounds__(1024)
select_block_scan_kernel(const int32_t* __restrict__ blk_cnt, int64_t nblk, int64_t* __restrict__ blk_off)
{
    __shared__ int64_t s_w[2][32];
    __shared__ int64_t s_carry[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { s_carry[0] = 0; s_carry[1] = 0; }
    __syncthreads();
    for (int64_t base = 0; base < nblk; base += 1024) {
        const int64_t b = base + threadIdx.x;
        int64_t v[2] = {0, 0};
        if (b < nblk) { v[0] = blk_cnt[2 * b]; v[1] = blk_cnt[2 * b + 1]; }
        int64_t inc[2] = {v[0], v[1]};
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int64_t a0 = __shfl_up_sync(0xFFFFFFFFu, inc[0], o), a1 = __shfl_up_sync(0xFFFFFFFFu, inc[1], o);
            if (lane >= o) { inc[0] += a0; inc[1] += a1; }
        }
        if (lane == 31) { s_w[0][warp] = inc[0]; s_w[1][warp] = inc[1]; }
        __syncthreads();
        int64_t wo[2] = {0, 0};
        for (int w = 0; w < warp; ++w) { wo[0] += s_w[0][w]; wo[1] += s_w[1][w]; }
        const int64_t c0 = s_carry[0], c1 = s_carry[1];
        if (b < nblk) { blk_off[2 * b] = c0 + wo[0] + inc[0] - v[0]; blk_off[2 * b + 1] = c1 + wo[1] + inc[1] - v[1]; }
        __syncthreads();
        if (threadIdx.x == 1023) { s_carry[0] = c0 + wo[0] + inc[0]; s_carry[1] = c1 + wo[1] + inc[1]; }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(SEL_T)
select_write_kernel(const float* __restrict__ scores, int64_t N, const SelectState* __restrict__ state,
                    const int64_t* __restrict__ blk_off, int64_t* __restrict__ indices)
{
    __shared__ int s_gt[SEL_T / 32], s_eq[SEL_T / 32];
    const uint32_t T = state->prefix;
    const int64_t k_ties = state->k_rem;
    const int64_t base = (int64_t)blockIdx.x * SEL_CHUNK + threadIdx.x * SEL_EPT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
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
    int64_t gt_before = blk_off[2 * blockIdx.x] + igt - gt;
    int64_t eq_before = blk_off[2 * blockIdx.x + 1] + ieq - eq;
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

}  // namespace

size_t select_workspace_bytes(int64_t N)
{
    const int64_t nblk = sel_nblk(N > 0 ? N : 1);
    return 3 * 2048 * sizeof(uint32_t) + 256 + align_up((size_t)nblk * 2 * sizeof(int64_t), 256) +
           align_up((size_t)nblk * 2 * sizeof(int32_t), 256);
}

cudaError_t launch_select_topk(const float* scores, int64_t N, int64_t k, int64_t* indices, void* ws,
                               cudaStream_t st)
{
    if (N == 0 || k == 0) return cudaSuccess;
    SelectWs w = carve(ws, N);
    cudaError_t e = cudaMemsetAsync(w.hist, 0, 3 * 2048 * sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    int64_t hb = (N / 4 + SEL_T - 1) / SEL_T;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (hb > cap) hb = cap;
    if (hb < 1) hb = 1;
    select_hist_kernel<0><<<(unsigned)hb, SEL_T, 0, st>>>(scores, N, w.state, w.hist);
    select_scan_kernel<0><<<1, 1024, 0, st>>>(w.hist, w.state, k);
    select_hist_kernel<1><<<(unsigned)hb, SEL_T, 0, st>>>(scores, N, w.state, w.hist + 2048);
    select_scan_kernel<1><<<1, 1024, 0, st>>>(w.hist + 2048, w.state, k);
    select_hist_kernel<2><<<(unsigned)hb, SEL_T, 0, st>>>(scores, N, w.state, w.hist + 4096);
    select_scan_kernel<2><<<1, 1024, 0, st>>>(w.hist + 4096, w.state, k);
    const int64_t nblk = sel_nblk(N);
    select_count_kernel<<<(unsigned)nblk, SEL_T, 0, st>>>(scores, N, w.state, w.blk_cnt);
    select_block_scan_kernel<<<1, 1024, 0, st>>>(w.blk_cnt, nblk, w.blk_off);
    select_write_kernel<<<(unsigned)nblk, SEL_T, 0, st>>>(scores, N, w.state, w.blk_off, indices);
    count_launches(9);
    return cudaGetLastError();
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
