// Adam prologue (Gamma) and the stand-alone generator of projection-matrix entries.
#include "qless_kernels.h"

namespace qless {

// Gamma_j = m'/(sqrt(v')+eps), m' = b1 m + (1-b1) g, v' = b2 v + (1-b2) g^2, every operation a
// separately rounded IEEE fp32 operation (no fused multiply-add), result rounded to bf16 (RNE).
// bm = fl(b1 m), bv = fl(b2 v) are passed in because they are the same for every row of the batch.
//
// The IEEE square root and division are the expensive part, and the result only keeps 8 bits. So the
// quotient is first formed with the approximate reciprocal-square-root unit (a few ulp of error); unless that value
// lies close to a bf16 rounding boundary (or outside the normal range) its bf16 rounding is already the one
// the exact sequence gives, and the exact sequence runs only for the rare remaining elements.

// Elements the fast path below gave up on (about one in a thousand on typical moments; all of them where
// eps / sqrt(v') is not small). Not inlined: it is long and the kernel holds 16 call sites. Without bias correction
// (c1 = c2 = 1) a second approximation is tried first, good for any eps / sqrt(v'): sqrt(v') as v' rs, the quotient
// by the approximate reciprocal (two special-function operations, a few ulp of error), accepted under the same two
// tests as the fast path; what is left takes the exact sequence.
__device__ __noinline__ float adam_dir_slow(float g, float bm, float bv, float omb1, float omb2, float eps, float c1, float c2)
{
    float m1 = __fadd_rn(bm, __fmul_rn(omb1, g));
    float v1 = __fadd_rn(bv, __fmul_rn(omb2, __fmul_rn(g, g)));
    if (c1 == 1.0f && c2 == 1.0f) {
        float rs, rc;
        asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(rs) : "f"(v1));
        const float den_a = __fadd_rn(__fmul_rn(v1, rs), eps);          // v1 = 0 gives NaN: fails the range test
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc) : "f"(den_a));
        const float q = __fmul_rn(m1, rc);
        const uint32_t qb = __float_as_uint(q);
        const bool in_range = (((qb >> 23) & 0xFFu) - 28u) <= 198u;
        const bool off_tie = ((qb - 0x7FE0u) & 0xFFFFu) > 0x40u;
        if (in_range && off_tie) return q;
    } else {
        m1 = __fdiv_rn(m1, c1); v1 = __fdiv_rn(v1, c2);                 // bias correction
    }
    const float den = __fadd_rn(__fsqrt_rn(v1), eps);
    return __fdiv_rn(m1, den);
}

// Fast path (no bias correction): one special-function operation per element (the kernel is bound by instruction
// issue, then by that unit at 16 lanes per clock per SM). v' is a sum of non-negative terms, so forming it with one
// fused multiply-add moves it by an ulp; m' may cancel and keeps the exact roundings. With rs = 1 / sqrt(v'),
// 1 / (sqrt(v') + eps) = rs / (1 + t), t = eps rs, and for t < 2^-8 the series 1 - t + t^2 is within t^3 < 2^-24 of
// 1 / (1 + t): q = u - u (t - t^2), u = m' rs. All roundings and the unit's error (2^-22.9) add up to less than 7 fp32
// ulps between this quotient and the exact sequence's, 13 steps of its significand.
// ok: t is small (a larger one, v' tiny or zero, rs huge or infinite, t possibly NaN, fails the test), q is well inside
// the normal range (biased exponent in [28, 226]: zeros, subnormals, infinities and NaNs all fall outside; so does
// every case in which rs or a product left the normal range, since q is then 0, infinite or NaN) and its low 16 bits
// are more than 32 away from the bf16 tie 0x8000. Then q rounds to the same bf16 as the exact quotient.
__device__ __forceinline__ float adam_dir_fast(float g, float bm, float bv, const AdamParams& ap, bool& ok)
{
    const float m1 = __fadd_rn(bm, __fmul_rn(ap.omb1, g));
    const float v1f = fmaf(ap.omb2, __fmul_rn(g, g), bv);
    float rs;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(rs) : "f"(v1f));
    const float t = ap.eps * rs;
    const float u = m1 * rs;
    const float q = fmaf(-u, fmaf(-t, t, t), u);
    const uint32_t qb = __float_as_uint(q);
    const bool in_range = (qb * 2u - (28u << 24)) <= ((198u << 24) | 0xFFFFFFu);
    const bool off_tie = ((qb << 16) - (0x7FE0u << 16)) > (0x40u << 16);
    ok = (t < 0.00390625f) & in_range & off_tie;          // no short circuit: three compares, no branch
    return q;
}

// Two neighbouring elements share one branch to the slow path.
__device__ __forceinline__ void adam_dir2(float& g0, float& g1, float bm0, float bm1, float bv0, float bv1, const AdamParams& ap)
{
    bool ok0 = false, ok1 = false;
    float q0 = 0.0f, q1 = 0.0f;
    if (!ap.bias_correct) { q0 = adam_dir_fast(g0, bm0, bv0, ap, ok0); q1 = adam_dir_fast(g1, bm1, bv1, ap, ok1); }
    if (!(ok0 & ok1)) {
        const float c1 = ap.bias_correct ? ap.c1 : 1.0f, c2 = ap.bias_correct ? ap.c2 : 1.0f;
        if (!ok0) q0 = adam_dir_slow(g0, bm0, bv0, ap.omb1, ap.omb2, ap.eps, c1, c2);
        if (!ok1) q1 = adam_dir_slow(g1, bm1, bv1, ap.omb1, ap.omb2, ap.eps, c1, c2);
    }
    g0 = q0; g1 = q1;
}

// One thread handles 8 consecutive columns (16-byte bf16 accesses); AG_ROWS is the number of consecutive
// rows whose loads it issues together.
constexpr int AG_ROWS = 4;

template <bool BF16_IN, bool ADAM, bool TILED>
__global__ void __launch_bounds__(256, 4)
adam_gamma_kernel(const void* __restrict__ grads, int64_t n, int64_t ld, const float* __restrict__ m,
                  const float* __restrict__ v, AdamParams ap, int64_t P, __nv_bfloat16* __restrict__ gamma)
{
    // A thread owns 8 consecutive coordinates and walks down all n rows, AG_ROWS at a time: the moments of its
    // coordinates are read from memory once per batch and stay in registers.
    const int64_t groups_per_row = P >> 3;
    for (int64_t cg = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; cg < groups_per_row;
         cg += (int64_t)gridDim.x * blockDim.x) {
        const int64_t j0 = cg << 3;
        float mm[8], vv[8];
        if (ADAM) {
            const float4 m0 = __ldcs(reinterpret_cast<const float4*>(m + j0)), m1 = __ldcs(reinterpret_cast<const float4*>(m + j0 + 4));
            const float4 v0 = __ldcs(reinterpret_cast<const float4*>(v + j0)), v1 = __ldcs(reinterpret_cast<const float4*>(v + j0 + 4));
            mm[0] = m0.x; mm[1] = m0.y; mm[2] = m0.z; mm[3] = m0.w; mm[4] = m1.x; mm[5] = m1.y; mm[6] = m1.z; mm[7] = m1.w;
            vv[0] = v0.x; vv[1] = v0.y; vv[2] = v0.z; vv[3] = v0.w; vv[4] = v1.x; vv[5] = v1.y; vv[6] = v1.z; vv[7] = v1.w;
#pragma unroll
            for (int k = 0; k < 8; ++k) { mm[k] = __fmul_rn(ap.beta1, mm[k]); vv[k] = __fmul_rn(ap.beta2, vv[k]); }
        }
        // TILED: [K block of 64 columns][row][64] so that a (256 rows x 64 columns) operand tile is one
        // contiguous 32 KiB span; otherwise plain row-major [n, P].
        __nv_bfloat16* out = TILED ? gamma + (((j0 >> 6) * n) << 6) + (j0 & 63) : gamma + j0;
        const int64_t out_ld = TILED ? 64 : P;
#pragma unroll 1
        for (int64_t row0 = 0; row0 < n; row0 += AG_ROWS) {
            // issue every row's loads before any arithmetic (memory-level parallelism)
            uint4 raw[AG_ROWS][BF16_IN ? 1 : 2];
#pragma unroll
            for (int r = 0; r < AG_ROWS; ++r) {
                if (row0 + r < n) {
                    if (BF16_IN) {
                        raw[r][0] = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(grads) + (row0 + r) * ld + j0));
                    } else {
                        const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(grads) + (row0 + r) * ld + j0);
                        raw[r][0] = __ldcs(p);
                        raw[r][BF16_IN ? 0 : 1] = __ldcs(p + 1);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < AG_ROWS; ++r) {
                const int64_t row = row0 + r;
                if (row >= n) break;
                float g[8];
                if (BF16_IN) {
                    const uint32_t w[4] = {raw[r][0].x, raw[r][0].y, raw[r][0].z, raw[r][0].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        g[2 * k] = __uint_as_float(w[k] << 16);
                        g[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
                    }
                } else {
                    const uint4 a = raw[r][0], b = raw[r][BF16_IN ? 0 : 1];
                    g[0] = __uint_as_float(a.x); g[1] = __uint_as_float(a.y); g[2] = __uint_as_float(a.z); g[3] = __uint_as_float(a.w);
                    g[4] = __uint_as_float(b.x); g[5] = __uint_as_float(b.y); g[6] = __uint_as_float(b.z); g[7] = __uint_as_float(b.w);
                }
                if (ADAM) {
#pragma unroll
                    for (int k = 0; k < 8; k += 2) adam_dir2(g[k], g[k + 1], mm[k], mm[k + 1], vv[k], vv[k + 1], ap);
                }
                uint32_t o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const __nv_bfloat162 pr = __floats2bfloat162_rn(g[2 * k], g[2 * k + 1]);
                    o[k] = *reinterpret_cast<const uint32_t*>(&pr);
                }
                *reinterpret_cast<uint4*>(out + row * out_ld) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
}

cudaError_t launch_adam_gamma(const void* grads, qless_dtype dtype, int64_t n, int64_t ld, const float* m,
                              const float* v, const AdamParams& ap, int64_t P, __nv_bfloat16* gamma,
                              bool tiled, cudaStream_t st)
{
    if (n == 0 || P == 0) return cudaSuccess;
    const int64_t total = P >> 3;          // a thread per group of 8 coordinates
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    const bool adam = (m != nullptr);
#define QLESS_AG(B, A, T) adam_gamma_kernel<B, A, T><<<(unsigned)blocks, threads, 0, st>>>(grads, n, ld, m, v, ap, P, gamma)
    const bool bf = (dtype == QLESS_BF16);
    if (bf && adam && tiled) QLESS_AG(true, true, true);
    else if (bf && adam) QLESS_AG(true, true, false);
    else if (bf && tiled) QLESS_AG(true, false, true);
    else if (bf) QLESS_AG(true, false, false);
    else if (adam && tiled) QLESS_AG(false, true, true);
    else if (adam) QLESS_AG(false, true, false);
    else if (tiled) QLESS_AG(false, false, true);
    else QLESS_AG(false, false, false);
#undef QLESS_AG
    count_launches(1);
    return cudaGetLastError();
}

// out[a][b] = sign(r0 + a, j0 + b) as int8.
__global__ void philox_entries_kernel(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj,
                                      int8_t* __restrict__ out)
{
    const int64_t total = nr * nj;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t a = idx / nj, b = idx - a * nj;
        const uint64_t j = (uint64_t)(j0 + b);
        uint32_t w[4];
        rademacher_block(seed, (uint32_t)(r0 + a), (uint32_t)(j >> 7), w);
        const uint32_t t = (uint32_t)(j & 127u);
        out[idx] = (int8_t)rademacher_sign_of(w[t >> 5], (int)(t & 31u));
    }
}

cudaError_t launch_philox_entries(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj, int8_t* out,
                                  cudaStream_t st)
{
    const int64_t total = nr * nj;
    if (total == 0) return cudaSuccess;
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    philox_entries_kernel<<<(unsigned)blocks, 256, 0, st>>>(seed, r0, nr, j0, nj, out);
    count_launches(1);
    return cudaGetLastError();
}

// out[a][b] = z(r0 + a, j0 + b) of the Gaussian matrix, as fp32 (values are bf16-representable). One thread per
// group of four columns; j0 is a multiple of 4.
__global__ void gaussian_entries_kernel(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj,
                                        float* __restrict__ out)
{
    const int64_t quads = (nj + 3) / 4;
    const int64_t total = nr * quads;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t a = idx / quads, b = idx - a * quads;
        const uint64_t q = (uint64_t)(j0 >> 2) + (uint64_t)b;
        uint32_t lo, hi;
        gaussian_quad_bf16x2(seed, (uint32_t)(r0 + a), (uint32_t)q, (uint32_t)(q >> 32), lo, hi);
        const float z[4] = {__uint_as_float(lo << 16), __uint_as_float(lo & 0xFFFF0000u),
                            __uint_as_float(hi << 16), __uint_as_float(hi & 0xFFFF0000u)};
        for (int t = 0; t < 4; ++t)
            if (4 * b + t < nj) out[a * nj + 4 * b + t] = z[t];
    }
}

cudaError_t launch_gaussian_entries(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj, float* out,
                                    cudaStream_t st)
{
    const int64_t total = nr * ((nj + 3) / 4);
    if (total == 0) return cudaSuccess;
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    gaussian_entries_kernel<<<(unsigned)blocks, 256, 0, st>>>(seed, r0, nr, j0, nj, out);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace qless
