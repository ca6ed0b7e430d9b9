// Projection (Eq. 1) on the CUDA cores: a plain tiled kernel used for shapes the tensor-core kernel
// does not take. part[s][i][r] = sum_{j in chunk s} Gamma[i][j] * sign(r, j).
#include "qless_kernels.h"

namespace qless {

namespace {

constexpr int PS_DR = 64;     // projected rows per block
constexpr int PS_GR = 32;     // gradient rows per block
constexpr int PS_T = 256;

template <bool GAUSS>
__global__ void __launch_bounds__(PS_T)
project_simt_kernel(const __nv_bfloat16* __restrict__ gamma, int64_t n, int64_t P, int32_t d,
                    int64_t chunk, uint32_t kblk_base, uint64_t seed, float* __restrict__ part)
{
    __shared__ __align__(16) float s_g[PS_GR][128];
    const int tid = threadIdx.x;
    const int tr = tid & (PS_DR - 1), ti = tid >> 6;           // ti = 0..3, 8 gradient rows each
    const uint32_t r = blockIdx.x * PS_DR + tr;
    const int64_t i0 = (int64_t)blockIdx.y * PS_GR;
    const int64_t k0 = (int64_t)blockIdx.z * chunk;
    const int64_t k1 = min(P, k0 + chunk);
    float acc[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) acc[u] = 0.0f;

    for (int64_t kb = k0; kb < k1; kb += 128) {
        __syncthreads();
        // 32 rows x 128 columns of Gamma -> fp32 in shared memory (rows >= n read as zero)
        for (int e = tid; e < PS_GR * 64; e += PS_T) {
            const int row = e >> 6, cp = e & 63;
            float2 f = make_float2(0.f, 0.f);
            if (i0 + row < n) {
                const int64_t j = kb + 2 * cp;     // tiled layout [P/64][n][64]
                const uint32_t w = *reinterpret_cast<const uint32_t*>(gamma + ((((j >> 6) * n + (i0 + row)) << 6) + (j & 63)));
                f.x = __uint_as_float(w << 16);
                f.y = __uint_as_float(w & 0xFFFF0000u);
            }
            *reinterpret_cast<float2*>(&s_g[row][2 * cp]) = f;
        }
        __syncthreads();
        const uint32_t blk = kblk_base + (uint32_t)(kb >> 7);
        uint32_t w[4];
        if (!GAUSS) rademacher_block(seed, r, blk, w);
#pragma unroll
        for (int wi = 0; wi < 4; ++wi) {
#pragma unroll 2
            for (int q = 0; q < 8; ++q) {               // 4 columns at a time
                if (GAUSS) {
                    uint32_t lo, hi;
                    gaussian_quad_bf16x2(seed, r, (blk << 5) | (uint32_t)(wi * 8 + q), blk >> 27, lo, hi);
                    const float z0 = __uint_as_float(lo << 16), z1 = __uint_as_float(lo & 0xFFFF0000u);
                    const float z2 = __uint_as_float(hi << 16), z3 = __uint_as_float(hi & 0xFFFF0000u);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const float4 g = *reinterpret_cast<const float4*>(&s_g[ti * 8 + u][wi * 32 + q * 4]);
                        acc[u] = fmaf(g.x, z0, acc[u]);
                        acc[u] = fmaf(g.y, z1, acc[u]);
                        acc[u] = fmaf(g.z, z2, acc[u]);
                        acc[u] = fmaf(g.w, z3, acc[u]);
                    }
                } else {
                    uint32_t sm[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int u = q * 4 + c;
                        const int beta = 15 - (u >> 1) + 16 * (u & 1);
                        sm[c] = ((w[wi] >> beta) & 1u) << 31;
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const float4 g = *reinterpret_cast<const float4*>(&s_g[ti * 8 + u][wi * 32 + q * 4]);
                        acc[u] += __uint_as_float(__float_as_uint(g.x) ^ sm[0]);
                        acc[u] += __uint_as_float(__float_as_uint(g.y) ^ sm[1]);
                        acc[u] += __uint_as_float(__float_as_uint(g.z) ^ sm[2]);
                        acc[u] += __uint_as_float(__float_as_uint(g.w) ^ sm[3]);
                    }
                }
            }
        }
    }
    float* out = part + (int64_t)blockIdx.z * n * d;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int64_t i = i0 + ti * 8 + u;
        if (i < n) out[i * d + r] = acc[u];
    }
}

}  // namespace

ProjectPlan plan_projection(int64_t n, int64_t P, int32_t d)
{
    // K-chunk length: a power of two in [1024, 262144] (so every chunk starts on a Philox block and a chain
    // of fp32 accumulations never exceeds 16384 tensor-core steps: with random signs its rounding error is about
    // 2^-24 sqrt(16384) = 8e-6 of the sum), the largest that still gives every SM about four work items of (256
    // gradient rows x 128 projected coordinates x chunk). Longer chunks mean fewer accumulator drains and fewer
    // partial sums to write and re-read: 65536 -> 262144 columns took 2.5 % off a 256 x 2^23 batch.
    ProjectPlan pl;
    pl.n = n; pl.P = P; pl.d = d; pl.k_base = 0; pl.gaussian = false;
    const int64_t tiles = (int64_t)(d / 128) * ((n + 255) / 256);
    int64_t chunk = 262144;
    while (chunk > 1024 && tiles * ((P + chunk - 1) / chunk) < 4 * (int64_t)sm_count()) chunk >>= 1;
    if (chunk > P) chunk = P;
    pl.chunk = chunk;
    pl.num_chunks = (int32_t)((P + chunk - 1) / chunk);
    return pl;
}

cudaError_t launch_project_simt(const __nv_bfloat16* gamma, const ProjectPlan& pl, uint64_t seed,
                                float* part, cudaStream_t st)
{
    if (pl.n == 0) return cudaSuccess;
    dim3 grid((unsigned)(pl.d / PS_DR), (unsigned)((pl.n + PS_GR - 1) / PS_GR), (unsigned)pl.num_chunks);
    if (pl.gaussian)
        project_simt_kernel<true><<<grid, PS_T, 0, st>>>(gamma, pl.n, pl.P, pl.d, pl.chunk, (uint32_t)(pl.k_base >> 7), seed, part);
    else
        project_simt_kernel<false><<<grid, PS_T, 0, st>>>(gamma, pl.n, pl.P, pl.d, pl.chunk, (uint32_t)(pl.k_base >> 7), seed, part);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace qless
