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
//       3 = int8 A in tensor memory; 4 = int8 A,B in shared memory in the shape the 8-bit scoring kernel issues
//       for 448 validation vectors (pair only): per K step one MMA of N = 256 and one of N = 192 on the same A;
//       5 = e2m1 (kind::mxf4, unit scale factors, 64 codes per MMA) A,B in shared memory in the same two-MMA shape, as the
//       2- and 1-bit scoring kernel issues them (pair only); 6 = e2m1 with A in tensor memory, N = 256 (pair only).
// PAIR: 0 = one CTA per 128 x 256 tile; 1 = CTA pair per 256 x 256 tile (cta_group::2).
template <int KIND, int PAIR>
__global__ void __launch_bounds__(128, 1)
mma_peak_kernel(int iters, unsigned int* timeout_word)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int A_BYTES = 128 * 128;                      // 128 rows x 128 bytes (one swizzle panel)
    constexpr int B_BYTES = ((KIND == 4 || KIND == 5) ? 224 : PAIR ? 128 : 256) * 128;
    constexpr uint32_t SF_COL = 448;                        // e2m1 kinds: 16 columns of unit scale factors (0x7F in every byte)
    uint8_t* sA = smem;
    uint8_t* sB = smem + A_BYTES;
    MbBars* bars = reinterpret_cast<MbBars*>(sB + B_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;

    for (int i = threadIdx.x; i < (A_BYTES + B_BYTES) / 4; i += blockDim.x)
        reinterpret_cast<uint32_t*>(smem)[i] = (KIND >= 5) ? ((i & 1) ? 0x2AA2A22Au : 0xA22A2AA2u)      // e2m1 codes +-1
                                               : (KIND >= 2) ? (0x01FF02FEu ^ (uint32_t)(i * 0x01010101u & 0x03030303u))
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
    if (KIND >= 5) {
        uint32_t v[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = 0x7F7F7F7Fu;
        tmem_st_x16(tmem_base + ((uint32_t)(warp * 32) << 16) + SF_COL, v);
        tmem_wait_st();
        tc_fence_before();
    }
    if (KIND == 1 || KIND == 3 || KIND == 6) {              // A operand: 64 columns (bf16 +-1.0 pairs, small int8, or e2m1 +-1) in every lane
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + 256;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t v[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = (KIND == 6) ? (((lane + k) & 1) ? 0x2AA2A22Au : 0xA22A2AA2u)
                                                : (KIND == 3) ? (0x01FF02FEu ^ (uint32_t)((lane + k) & 3) * 0x01010101u)
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
        const uint32_t idesc192 = make_idesc(2, 1, 1, M, 192);
        const uint64_t adesc = make_smem_desc_sw128(smem_u32(sA));
        const uint64_t bdesc = make_smem_desc_sw128(smem_u32(sB));
        const uint64_t bdesc192 = make_smem_desc_sw128(smem_u32(sB + 128 * 128));    // this CTA's 96 rows of the second MMA
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
                } else if (KIND == 5) {
                    if (PAIR) {
                        mma_mxf4_ss_pair(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), make_idesc_mxf4(256, 256), tmem_base + SF_COL, acc);
                        mma_mxf4_ss_pair(tmem_base + 256, adesc + (uint64_t)(2 * k), bdesc192 + (uint64_t)(2 * k), make_idesc_mxf4(256, 192), tmem_base + SF_COL, acc);
                    }
                } else if (KIND == 6) {
                    if (PAIR) mma_mxf4_ts_pair(tmem_base, tmem_base + 256 + 8 * k, bdesc + (uint64_t)(2 * k), make_idesc_mxf4(256, 256), tmem_base + SF_COL, acc);
                } else if (KIND == 4) {
                    if (PAIR) {
                        mma_i8_ss_pair(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, acc);
                        mma_i8_ss_pair(tmem_base + 256, adesc + (uint64_t)(2 * k), bdesc192 + (uint64_t)(2 * k), idesc192, acc);
                    }
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

// L2 -> shared memory streaming rate of TMA alone: every CTA keeps TS_STAGES stages of three 128-row x 128-byte
// boxes (48 KiB, the operand bytes of one K block of 8-bit scoring, rounded up) in flight from a buffer of
// 512 rows x 8192 bytes that stays in L2, and nothing consumes them.
constexpr int TS_STAGES = 4;
constexpr int TS_BOX = 128 * 128;
struct __align__(8) TsBars { uint64_t full[TS_STAGES]; uint32_t abort_flag; };

__global__ void __launch_bounds__(128, 1)
tma_stream_kernel(const __grid_constant__ CUtensorMap tmap, int iters, unsigned int* timeout_word)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    TsBars* bars = reinterpret_cast<TsBars*>(smem + (size_t)TS_STAGES * 3 * TS_BOX);
    if (threadIdx.x == 0) {
        for (int s = 0; s < TS_STAGES; ++s) mbar_init(smem_u32(&bars->full[s]), 1);
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = true;
        uint32_t tile = blockIdx.x * 7u;
        for (int it = 0; it < iters && ok; ++it) {
            const int s = it % TS_STAGES;
            const uint32_t bar = smem_u32(&bars->full[s]);
            if (it >= TS_STAGES) ok = mbar_wait(bar, (uint32_t)(it / TS_STAGES - 1) & 1u, &bars->abort_flag, timeout_word, TO_PRODUCER);
            if (!ok) break;
            mbar_arrive_expect_tx(bar, 3 * TS_BOX);
#pragma unroll
            for (int b = 0; b < 3; ++b, ++tile)
                tma_load_3d(smem_u32(smem + (size_t)(s * 3 + b) * TS_BOX), &tmap, bar, (int32_t)(tile & 63u) * 128,
                            (int32_t)((tile >> 6) & 3u) * 128, 0);
        }
        // every armed stage lands before the CTA leaves (bounded)
        const int issued = ok ? iters : 0;
        for (int it = (issued > TS_STAGES ? issued - TS_STAGES : 0); it < issued; ++it)
            mbar_wait(smem_u32(&bars->full[it % TS_STAGES]), (uint32_t)(it / TS_STAGES) & 1u, &bars->abort_flag, timeout_word, TO_PRODUCER);
        if (!ok)
            for (int s = 0; s < TS_STAGES; ++s)
                for (uint32_t t = 0; t < (1u << 16); ++t)
                    if (mbar_try_wait(smem_u32(&bars->full[s]), 0) || mbar_try_wait(smem_u32(&bars->full[s]), 1)) break;
    }
    __syncthreads();
}

// The two together, as 8-bit scoring runs them: the leader of a CTA pair issues the int8 MMAs of one K block
// (4 K steps x (N = 256, N = 192), operands resident in shared memory) back to back and commits once per K block;
// in both CTAs a second thread streams one 48 KiB stage per K block from L2 into other shared memory, MX_STAGES
// ahead, re-arming a stage when the commit of the K block that "used" it has arrived. The MMAs never wait for
// data: what this measures is how much the copies landing in shared memory slow the tensor pipe's operand reads.
constexpr int MX_STAGES = 3;
struct __align__(8) MxBars { uint64_t done, full[MX_STAGES], empty[MX_STAGES]; uint32_t tmem_base; uint32_t abort_flag; };

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1)
mma_tma_mix_kernel(const __grid_constant__ CUtensorMap tmap, int iters, int with_copies, unsigned int* timeout_word)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int A_BYTES = 128 * 128, B_BYTES = 224 * 128;
    uint8_t* sA = smem;
    uint8_t* sB = smem + A_BYTES;
    uint8_t* sS = smem + A_BYTES + 32 * 1024;               // stream stages, 1 KiB aligned
    MxBars* bars = reinterpret_cast<MxBars*>(sS + (size_t)MX_STAGES * 3 * TS_BOX);
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = cluster_ctarank();

    for (int i = threadIdx.x; i < (A_BYTES + B_BYTES) / 4; i += blockDim.x)
        reinterpret_cast<uint32_t*>(smem)[i] = 0x01FF02FEu ^ (uint32_t)(i * 0x01010101u & 0x03030303u);
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars->done), 1);
        for (int s = 0; s < MX_STAGES; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->empty[s]), 1); }
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap);
    }
    if (warp == 0) { tmem_alloc_pair(smem_u32(&bars->tmem_base), 512); tmem_relinquish_pair(); }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (threadIdx.x == 0 && rank == 0) {
        const uint32_t idesc = make_idesc(2, 1, 1, 256, 256), idesc192 = make_idesc(2, 1, 1, 256, 192);
        const uint64_t adesc = make_smem_desc_sw128(smem_u32(sA));
        const uint64_t bdesc = make_smem_desc_sw128(smem_u32(sB));
        const uint64_t bdesc192 = make_smem_desc_sw128(smem_u32(sB + 128 * 128));
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t acc = (it > 0 || k > 0) ? 1u : 0u;
                mma_i8_ss_pair(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, acc);
                mma_i8_ss_pair(tmem_base + 256, adesc + (uint64_t)(2 * k), bdesc192 + (uint64_t)(2 * k), idesc192, acc);
            }
            mma_commit_pair(smem_u32(&bars->empty[it % MX_STAGES]));      // arrives in both CTAs
        }
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bars->done)) : "memory");
        mbar_wait(smem_u32(&bars->done), 0, &bars->abort_flag, timeout_word, TO_MMA);
    } else if (threadIdx.x == 32 && with_copies) {
        bool ok = true;
        uint32_t tile = blockIdx.x * 7u;
        int issued = 0;
        for (int it = 0; it < iters && ok; ++it) {
            const int s = it % MX_STAGES;
            const uint32_t bar = smem_u32(&bars->full[s]);
            if (it >= MX_STAGES) {
                const uint32_t par = (uint32_t)(it / MX_STAGES - 1) & 1u;
                ok = mbar_wait_cluster(smem_u32(&bars->empty[s]), par, &bars->abort_flag, timeout_word, TO_PRODUCER) &&
                     mbar_wait(bar, par, &bars->abort_flag, timeout_word, TO_PRODUCER);
                if (!ok) break;
            }
            mbar_arrive_expect_tx(bar, 3 * TS_BOX);
#pragma unroll
            for (int b = 0; b < 3; ++b, ++tile)
                tma_load_3d(smem_u32(sS + (size_t)(s * 3 + b) * TS_BOX), &tmap, bar, (int32_t)(tile & 63u) * 128,
                            (int32_t)((tile >> 6) & 3u) * 128, 0);
            ++issued;
        }
        // every armed stage lands before the CTA leaves (bounded)
        for (int it = (issued > MX_STAGES ? issued - MX_STAGES : 0); it < issued; ++it)
            if (!mbar_wait(smem_u32(&bars->full[it % MX_STAGES]), (uint32_t)(it / MX_STAGES) & 1u, &bars->abort_flag, timeout_word, TO_PRODUCER)) break;
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// The int8 tensor pipe on operands that change: the leader of a CTA pair issues the MMAs of 8-bit scoring at 448
// validation vectors (per K block four K steps of one N = 256 and one N = 192 MMA on the same A), and every K block
// reads a stage that TMA has just brought from a 4 MiB buffer the caller filled with pseudo-random int8 values (256
// distinct 16 KiB boxes, taken in a sequence that differs from CTA to CTA), MC_STAGES stages ahead. TMA streams four
// times faster than the MMAs consume (micro-benchmark 9), so in steady state the MMAs never wait: what this adds to
// micro-benchmark 8 is data that toggles the operand paths, i.e. the power the tensor pipe draws on real codes, and
// with it the clock the power cap grants. The accumulator restarts every 64 K blocks, as a checkpoint of d = 8192 does.
constexpr int MC_STAGES = 4;
struct __align__(8) McBars { uint64_t done, full[MC_STAGES], empty[MC_STAGES]; uint32_t tmem_base; uint32_t abort_flag; };

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1)
mma_stream_consume_kernel(const __grid_constant__ CUtensorMap tmap, int iters, unsigned int* timeout_word)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int STAGE = 3 * TS_BOX;                       // A (128 rows) | B rows of the N = 256 MMA | B rows of the N = 192 MMA
    McBars* bars = reinterpret_cast<McBars*>(smem + (size_t)MC_STAGES * STAGE);
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = cluster_ctarank();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars->done), 1);
        for (int s = 0; s < MC_STAGES; ++s) { mbar_init(smem_u32(&bars->full[s]), 1); mbar_init(smem_u32(&bars->empty[s]), 1); }
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap);
    }
    if (warp == 0) { tmem_alloc_pair(smem_u32(&bars->tmem_base), 512); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (threadIdx.x == 0 && rank == 0) {
        const uint32_t idesc = make_idesc(2, 1, 1, 256, 256), idesc192 = make_idesc(2, 1, 1, 256, 192);
        bool ok = true;
        for (int it = 0; it < iters && ok; ++it) {
            const int s = it % MC_STAGES;
            ok = mbar_wait(smem_u32(&bars->full[s]), (uint32_t)(it / MC_STAGES) & 1u, &bars->abort_flag, timeout_word, TO_MMA);
            if (!ok) break;
            tc_fence_after();
            const uint32_t st = smem_u32(smem + (size_t)s * STAGE);
            const uint64_t adesc = make_smem_desc_sw128(st);
            const uint64_t bdesc = make_smem_desc_sw128(st + TS_BOX);
            const uint64_t bdesc192 = make_smem_desc_sw128(st + 2 * TS_BOX);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t acc = ((it & 63) > 0 || k > 0) ? 1u : 0u;
                mma_i8_ss_pair(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, acc);
                mma_i8_ss_pair(tmem_base + 256, adesc + (uint64_t)(2 * k), bdesc192 + (uint64_t)(2 * k), idesc192, acc);
            }
            mma_commit_pair(smem_u32(&bars->empty[s]));      // arrives in both CTAs
        }
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bars->done)) : "memory");
        mbar_wait_quiet(smem_u32(&bars->done), 0u);
    } else if (threadIdx.x == 32) {
        // both CTAs: this CTA's three boxes of every stage; all of a stage's bytes complete on the leader's barrier
        bool ok = true;
        uint32_t tile = blockIdx.x * 37u;
        uint32_t issued = 0;
        for (int it = 0; it < iters && ok; ++it) {
            const int s = it % MC_STAGES;
            if (it >= MC_STAGES) {
                ok = mbar_wait_cluster(smem_u32(&bars->empty[s]), (uint32_t)(it / MC_STAGES - 1) & 1u, &bars->abort_flag, timeout_word, TO_PRODUCER);
                if (!ok) break;
            }
            const uint32_t full = map_to_cta(smem_u32(&bars->full[s]), 0);
            if (rank == 0) mbar_arrive_expect_tx(smem_u32(&bars->full[s]), 2 * STAGE);
#pragma unroll
            for (int b = 0; b < 3; ++b, ++tile)
                tma_load_3d_pair(smem_u32(smem + (size_t)s * STAGE + (size_t)b * TS_BOX), &tmap, full, (int32_t)(tile & 63u) * 128,
                                 (int32_t)((tile >> 6) & 3u) * 128, 0);
            ++issued;
        }
        if (!ok && rank == 0)       // a failed wait: let the stages armed last land before the CTA leaves (bounded)
            for (uint32_t j = (issued > (uint32_t)MC_STAGES ? issued - MC_STAGES : 0u); j < issued; ++j)
                if (!mbar_wait_quiet(smem_u32(&bars->full[j % MC_STAGES]), (j / MC_STAGES) & 1u)) break;
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
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
        } else if ((what >= 3 && what <= 5) || what == 7 || what == 8 || what == 13 || what == 14) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(sms / 2 * 2)); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem; cfg.stream = st;
            cudaLaunchAttribute attr; attr.id = cudaLaunchAttributeClusterDimension; attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr; cfg.numAttrs = 1;
#define QLESS_MB_LAUNCH(K)                                                                                           \
            err = cudaFuncSetAttribute(mma_peak_kernel<K, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
            if (err == cudaSuccess) err = cudaLaunchKernelEx(&cfg, mma_peak_kernel<K, 1>, (int)iters, flag);
            if (what == 3) { QLESS_MB_LAUNCH(0) } else if (what == 4) { QLESS_MB_LAUNCH(1) } else if (what == 5) { QLESS_MB_LAUNCH(2) }
            else if (what == 7) { QLESS_MB_LAUNCH(3) } else if (what == 8) { QLESS_MB_LAUNCH(4) } else if (what == 13) { QLESS_MB_LAUNCH(5) }
            else { QLESS_MB_LAUNCH(6) }
#undef QLESS_MB_LAUNCH
            ops = (double)(sms / 2) * iters * 4.0 * 2.0 * 256 * ((what == 8 || what == 13) ? 448 : 256) *
                  (what >= 13 ? 64 : (what == 5 || what == 7 || what == 8) ? 32 : 16);
        } else if (what == 6) {
            const size_t need = (size_t)sms * 8 * 256 * sizeof(uint32_t);
            QLESS_REQUIRE(scratch != nullptr && scratch_bytes >= need, QLESS_ERR_WORKSPACE, "scratch of %zu bytes required", need);
            popc_peak_kernel<<<sms * 8, 256, 0, st>>>(iters, 12345u, reinterpret_cast<uint32_t*>(scratch));
            ops = (double)sms * 8 * 256 * iters * 32.0;           // word operations: one XOR + POPC + IADD each
        } else if (what == 9 || what == 10 || what == 11 || what == 12) {
            const size_t need = (size_t)512 * 8192;
            if (scratch == nullptr || scratch_bytes < need || (reinterpret_cast<uintptr_t>(scratch) % 16) != 0) {
                cudaEventDestroy(e0); cudaEventDestroy(e1);
                return fail(QLESS_ERR_WORKSPACE, "16-byte aligned scratch of %zu bytes required", need);
            }
            CUtensorMap tm;
            const qless_status ts = make_tmap_3d_u8(&tm, scratch, 8192, 512, 1, 8192, need, 128, 128, true);
            if (ts != QLESS_OK) { cudaEventDestroy(e0); cudaEventDestroy(e1); return ts; }
            if (what == 9) {
                const size_t ts_smem = 1024 + (size_t)TS_STAGES * 3 * TS_BOX + sizeof(TsBars);
                err = cudaFuncSetAttribute(tma_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ts_smem);
                if (err == cudaSuccess) tma_stream_kernel<<<sms, 128, ts_smem, st>>>(tm, iters, flag);
                ops = (double)sms * iters * 3.0 * TS_BOX;             // bytes moved from L2 into shared memory
            } else if (what == 12) {
                const size_t mc_smem = 1024 + (size_t)MC_STAGES * 3 * TS_BOX + sizeof(McBars);
                err = cudaFuncSetAttribute(mma_stream_consume_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mc_smem);
                if (err == cudaSuccess) mma_stream_consume_kernel<<<sms / 2 * 2, 128, mc_smem, st>>>(tm, iters, flag);
                ops = (double)(sms / 2) * iters * 4.0 * 2.0 * 256 * 448 * 32;
            } else {
                const size_t mx_smem = 1024 + 128 * 128 + 32 * 1024 + (size_t)MX_STAGES * 3 * TS_BOX + sizeof(MxBars);
                err = cudaFuncSetAttribute(mma_tma_mix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mx_smem);
                if (err == cudaSuccess) mma_tma_mix_kernel<<<sms / 2 * 2, 128, mx_smem, st>>>(tm, iters, what == 10 ? 1 : 0, flag);
                ops = (double)(sms / 2) * iters * 4.0 * 2.0 * 256 * 448 * 32;
            }
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
