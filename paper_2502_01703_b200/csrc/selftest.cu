// Self-test of the bounded device-side waits: a wait that nothing will ever satisfy must give up, record which
// role gave up in the device timeout word, make the other roles of its CTA leave their waits, and let the kernel
// return normally, so that the context stays usable and qless_check reports QLESS_ERR_TIMEOUT. The kernel uses the
// same mbar_wait the tensor-core kernels use, with the poll limit passed in; it touches no tensor memory and
// starts no copy.
#include "qless_kernels.h"
#include "tc_common.cuh"

namespace qless {

namespace {

using namespace tc;

__global__ void __launch_bounds__(64, 1)
selftest_timeout_kernel(uint32_t polls, unsigned int* timeout_word)
{
    __shared__ __align__(8) uint64_t bar[2];
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar[0]), 1);
        mbar_init(smem_u32(&bar[1]), 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    // thread 0 plays a producer whose slot is never released: it gives up after `polls` polls
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar[0]), 0u, &abort_flag, timeout_word, TO_PRODUCER, polls);
    // thread 32 plays a consumer with a far longer limit: it must leave as soon as it sees the CTA-wide abort flag,
    // without recording a code of its own
    if (threadIdx.x == 32) mbar_wait(smem_u32(&bar[1]), 0u, &abort_flag, timeout_word, TO_EPILOGUE, polls * 256u);
    __syncthreads();
}

}  // namespace

}  // namespace qless

using namespace qless;

extern "C" qless_status qless_selftest_timeout(int32_t polls, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(polls >= 256 && polls <= (1 << 16), QLESS_ERR_INVALID_ARG, "polls must be in [256, 65536] (polls=%d)", polls);
    unsigned int* flag = timeout_flag_ptr();
    QLESS_REQUIRE(flag != nullptr, QLESS_ERR_CUDA, "cannot resolve the device timeout flag");
    selftest_timeout_kernel<<<1, 64, 0, st>>>((uint32_t)polls, flag);
    count_launches(1);
    QLESS_CUDA_TRY(cudaGetLastError());
    return QLESS_OK;
}
