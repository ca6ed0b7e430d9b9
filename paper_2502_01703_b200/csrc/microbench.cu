// Peak-rate micro-benchmarks of the units the kernels are measured against and for which no vendor figure
// has been measured on this machine: back-to-back tcgen05.mma (bf16 and int8, one CTA or a CTA pair per
// tile, operands resident in shared/tensor memory) and the XOR + POPC + IADD instruction mix of 1-bit
// scoring. They do no useful work; operands are filled with a non-trivial bit pattern so that power draw
// is representative.
#include "qless_kernels.h"
#include "tc_common.cuh"

namespace qless {

namespace {

using namespace tc;

struct __align__(8) MbBars { uint64_t done; uint32_t tmem_base; uint32_t abort_flag; };

// KIND: 0 = bf16 A,B in shared memory; 1 = bf16 A in tensor memory; 2 = int8 A,B in shared memory;
//       3 = int8 A in tensor memory.
// PAIR: 0 = one CTA per 128 x 256 tile; 1 = CTA pair per 256 x 256 tile (cta_group::2).
template <int KIND, int PAIR>
__global__ void __launch_bounds__(128, 1)
mma_peak_kernel(int iters, unsigned int* timeout_word)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int A_BYTES = 128 * 128;                      // 128 rows x 128 bytes (one swizzle panel)
    constexpr int B_BYTES = (PAIR ? 128 : 256) * 128;
    uint8_t* sA = smem;
    uint8_t* sB = smem + A_BYTES;
    MbBars* bars = reinterpret_cast<MbBars*>(sB + B_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;

    for (int i = threadIdx.x; i < (A_BYTES + B_BYTES) / 4; i += blockDim.x)
        reinterpret_cast<uint32_t*>(smem)[i] = (KIND >= 2) ? (0x01FF02FEu ^ (uint32_t)(i * 0x01010101u & 0x03030303u))
                                                            : ((i & 1) ? 0x3F80BF80u : 0xBF803F80u);
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bars->done), 1); bars->abort_flag = 0; fence_barrier_init(); }
    if (warp == 0) {
        if (PAIR) { tmem_alloc_pair(smem_u32(&bars->tmem_base), 512); tmem_relinquish_pair(); }
        else { tmem_alloc(smem_u32(&bars->tmem_base), 512); tmem_relinquish(); }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    if (KIND == 1 || KIND == 3) {                           // A operand: 64 columns (bf16 +-1.0 pairs, or small int8) in every lane
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + 256;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t v[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = (KIND == 3) ? (0x01FF02FEu ^ (uint32_t)((lane + k) & 3) * 0x01010101u)
                                                            : (((lane + k) & 1) ? 0x3F80BF80u : 0xBF803F80u);
            tmem_st_x16(taddr + c * 16, v);
        }
        tmem_wait_st();
        tc_fence_before();
    }
    __syncthreads();
    if (PAIR) cluster_sync_all();
    tc_fence_after();

    if (threadIdx.x == 0 && rank == 0) {
        constexpr uint32_t M = PAIR ? 256 : 128;
        const uint32_t idesc = (KIND >= 2) ? make_idesc(2, 1, 1, M, 256) : make_idesc(1, 1, 1, M, 256);
        const uint64_t adesc = make_smem_desc_sw128(smem_u32(sA));
        const uint64_t bdesc = make_smem_desc_sw128(smem_u32(sB));
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {                   // four K steps of 32 bytes inside the 128-byte panel
                const uint32_t acc = (it > 0 || k > 0) ? 1u : 0u;
                if (KIND == 0) {
                    if (PAIR) asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                           ::"r"(tmem_base), "l"(adesc + (uint64_t)(2 * k)), "l"(bdesc + (uint64_t)(2 * k)), "r"(idesc), "r"(acc) : "memory");
                    else asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                      ::"r"(tmem_base), "l"(adesc + (uint64_t)(2 * k)), "l"(bdesc + (uint64_t)(2 * k)), "r"(idesc), "r"(acc) : "memory");
                } else if (KIND == 1) {
                    if (PAIR) mma_f16_ts_pair(tmem_base, tmem_base + 256 + 8 * k, bdesc + (uint64_t)(2 * k), idesc, acc);
                    else mma_f16_ts(tmem_base, tmem_base + 256 + 8 * k, bdesc + (uint64_t)(2 * k), idesc, acc);
                } else if (KIND == 3) {
                    if (PAIR) mma_i8_ts_pair(tmem_base, tmem_base + 256 + 8 * k, bdesc + (uint64_t)(2 * k), idesc, acc);
                } else {
                    if (PAIR) mma_i8_ss_pair(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, acc);
                    else mma_i8_ss(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, acc);
                }
            }
        }
        if (PAIR) asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bars->done)) : "memory");
        else mma_commit(smem_u32(&bars->done));
        mbar_wait(smem_u32(&bars->done), 0, &bars->abort_flag, timeout_word, TO_MMA);
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512);
    }
}

// 1-bit scoring instruction mix: acc += popc(a ^ b), 32 independent accumulators per thread.
__global__ void __launch_bounds__(256)
popc_peak_kernel(int iters, uint32_t seed, uint32_t* out)
{
    uint32_t a[4], b[8];
    int acc[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u) a[u] = seed * (threadIdx.x + 1) + u * 0x9E3779B9u;
#pragma unroll
    for (int w = 0; w < 8; ++w) b[w] = seed ^ (blockIdx.x * 2654435761u + w * 0x85EBCA6Bu);
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int w = 0; w < 8; ++w) acc[u][w] = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int w = 0; w < 8; ++w) acc[u][w] += __popc(a[u] ^ b[w]);
#pragma unroll
        for (int u = 0; u < 4; ++u) a[u] += 0x85EBCA6Bu;                       // new operands every iteration
#pragma unroll
        for (int w = 0; w < 8; ++w) b[w] += 0x9E3779B9u;
    }
    int s = 0;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int w = 0; w < 8; ++w) s += acc[u][w];
    out[blockIdx.x * blockDim.x + threadIdx.x] = (uint32_t)s;
}

}  // namespace

}  // namespace qless

using namespace qless;

extern "C" qless_status qless_microbench(int32_t what, int32_t iters, float* ms_out, double* ops_out, void* scratch,
                                         size_t scratch_bytes, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(ms_out != nullptr && ops_out != nullptr, QLESS_ERR_INVALID_ARG, "ms_out and ops_out (host) are required");
    QLESS_REQUIRE(iters > 0, QLESS_ERR_INVALID_ARG, "iters must be positive");
    const int sms = sm_count();
    unsigned int* flag = timeout_flag_ptr();
    QLESS_REQUIRE(flag != nullptr, QLESS_ERR_CUDA, "cannot resolve the device timeout flag");
    cudaEvent_t e0, e1;
    QLESS_CUDA_TRY(cudaEventCreate(&e0));
    QLESS_CUDA_TRY(cudaEventCreate(&e1));
    const size_t smem = 1024 + 128 * 128 + 256 * 128 + sizeof(MbBars);
    double ops = 0.0;
    cudaError_t err = cudaSuccess;
    for (int rep = 0; rep < 2 && err == cudaSuccess; ++rep) {        // first pass warms up
        QLESS_CUDA_TRY(cudaEventRecord(e0, st));
        if (what >= 0 && what <= 2) {
#define QLESS_MB_LAUNCH(K)                                                                                           \
            err = cudaFuncSetAttribute(mma_peak_kernel<K, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
            if (err == cudaSuccess) mma_peak_kernel<K, 0><<<sms, 128, smem, st>>>(iters, flag);
            if (what == 0) { QLESS_MB_LAUNCH(0) } else if (what == 1) { QLESS_MB_LAUNCH(1) } else { QLESS_MB_LAUNCH(2) }
#undef QLESS_MB_LAUNCH
            ops = (double)sms * iters * 4.0 * 2.0 * 128 * 256 * (what == 2 ? 32 : 16);
        } else if ((what >= 3 && what <= 5) || what == 7) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(sms / 2 * 2)); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem; cfg.stream = st;
            cudaLaunchAttribute attr; attr.id = cudaLaunchAttributeClusterDimension; attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr; cfg.numAttrs = 1;
#define QLESS_MB_LAUNCH(K)                                                                                           \
            err = cudaFuncSetAttribute(mma_peak_kernel<K, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
            if (err == cudaSuccess) err = cudaLaunchKernelEx(&cfg, mma_peak_kernel<K, 1>, (int)iters, flag);
            if (what == 3) { QLESS_MB_LAUNCH(0) } else if (what == 4) { QLESS_MB_LAUNCH(1) } else if (what == 5) { QLESS_MB_LAUNCH(2) } else { QLESS_MB_LAUNCH(3) }
#undef QLESS_MB_LAUNCH
            ops = (double)(sms / 2) * iters * 4.0 * 2.0 * 256 * 256 * (what == 5 || what == 7 ? 32 : 16);
        } else if (what == 6) {
            const size_t need = (size_t)sms * 8 * 256 * sizeof(uint32_t);
            QLESS_REQUIRE(scratch != nullptr && scratch_bytes >= need, QLESS_ERR_WORKSPACE, "scratch of %zu bytes required", need);
            popc_peak_kernel<<<sms * 8, 256, 0, st>>>(iters, 12345u, reinterpret_cast<uint32_t*>(scratch));
            ops = (double)sms * 8 * 256 * iters * 32.0;           // word operations: one XOR + POPC + IADD each
        } else {
            cudaEventDestroy(e0); cudaEventDestroy(e1);
            return fail(QLESS_ERR_INVALID_ARG, "unknown micro-benchmark %d", what);
        }
        if (err == cudaSuccess) err = cudaGetLastError();
        count_launches(1);
        QLESS_CUDA_TRY(cudaEventRecord(e1, st));
        QLESS_CUDA_TRY(cudaEventSynchronize(e1));
    }
    float ms = 0.f;
    if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    if (err != cudaSuccess) return cuda_fail(err, "micro-benchmark launch");
    *ms_out = ms; *ops_out = ops;
    return QLESS_OK;
}
