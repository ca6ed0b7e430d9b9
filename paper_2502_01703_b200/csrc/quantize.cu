// Stage 2: (sum of projection partials) -> L2 normalise (Eq. 2) -> absmax b-bit codes (Eq. 4-5) -> pack.
// HBM-bound: each row is read once (4*d bytes per partial) and d*b/8 + 8 bytes are written.
#include "qless_kernels.h"

namespace qless {

namespace {

constexpr int QT = 256;        // threads per row
constexpr int QMAX_V4 = 8;     // float4 chunks per thread  => d <= 256 * 8 * 4 = 8192

__device__ __forceinline__ double warp_sum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
    return x;
}
// x >= 0 and not NaN (a running fmaxf that starts at 0): such floats order like their bit patterns, so the
// warp-wide integer maximum (one instruction) is their maximum.
__device__ __forceinline__ float warp_max(float x)
{
    return __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(x)));
}
__device__ __forceinline__ int warp_sum_i(int x)
{
    return __reduce_add_sync(0xFFFFFFFFu, x);
}

// ABSMEAN: the scale comes from the mean absolute value of the row instead of its maximum (see the absmean
// branch below); BITS = 1 has no scale and is always instantiated with ABSMEAN = false. FULL: d = 8192, every
// thread owns eight whole float4 chunks and the per-chunk bounds tests compile away (the kernel is bound by
// instruction issue: those tests and the per-chunk tests of the call's options were a tenth of its instructions).
// MULTI: the row is the sum of num_parts > 1 partial rows (fewer resident blocks, more registers: eight loads in flight).
template <int BITS, bool ABSMEAN = false, bool FULL = false, bool MULTI = false>
__global__ void __launch_bounds__(QT, MULTI ? 3 : 5)
quantize_kernel(const float* __restrict__ parts, int32_t num_parts, float scale, int64_t n, int32_t d,
                int normalize, uint8_t* __restrict__ codes, float* __restrict__ scales,
                int32_t* __restrict__ sumsq, float* __restrict__ proj_out)
{
    __shared__ double s_d[QT / 32];
    __shared__ float s_f[QT / 32];
    __shared__ int s_i[QT / 32];
    __shared__ float s_par[3];            // the row's scalars: 1 / norm, scale S, multiplier of Eq. 5
    __shared__ __align__(16) uint8_t s_out[8192];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nv4 = d >> 2;                       // float4 chunks per row (multiple of 32)
    const int64_t part_stride = n * (int64_t)d;
    const int row_bytes = d * BITS / 8;

    for (int64_t row = blockIdx.x; row < n; row += gridDim.x) {
        // ask L2 for the row this CTA will take next, so that its loads find it there
        if (tid == 0 && row + gridDim.x < n) {
            for (int s = 0; s < num_parts; ++s)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(parts + s * part_stride + (row + gridDim.x) * d), "r"(d * 4) : "memory");
        }
        float4 x[QMAX_V4];
        // ---- load + fixed-order sum of partials (part 0, 1, 2, ... for every element), scaled once ----
        if (!MULTI) {
            const float4* p = reinterpret_cast<const float4*>(parts + row * d) + tid;
#pragma unroll
            for (int k = 0; k < QMAX_V4; ++k)
                x[k] = (FULL || tid + k * QT < nv4) ? __ldcs(p + k * QT) : make_float4(0.f, 0.f, 0.f, 0.f);
        } else {
            // many parts (the projection's K chunks), usually few rows: a thread keeps eight loads of one chunk's
            // column in flight and adds them in part order
            const int64_t ps4 = part_stride >> 2;
#pragma unroll
            for (int k = 0; k < QMAX_V4; ++k) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                if (FULL || tid + k * QT < nv4) {
                    const float4* p = reinterpret_cast<const float4*>(parts + row * d) + tid + k * QT;
                    a = __ldcs(p);
                    int s = 1;
                    for (; s + 8 <= num_parts; s += 8) {
                        float4 b[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) b[u] = __ldcs(p + (s + u) * ps4);
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            a.x = __fadd_rn(a.x, b[u].x); a.y = __fadd_rn(a.y, b[u].y);
                            a.z = __fadd_rn(a.z, b[u].z); a.w = __fadd_rn(a.w, b[u].w);
                        }
                    }
                    for (; s < num_parts; ++s) {
                        const float4 b = __ldcs(p + s * ps4);
                        a.x = __fadd_rn(a.x, b.x); a.y = __fadd_rn(a.y, b.y);
                        a.z = __fadd_rn(a.z, b.z); a.w = __fadd_rn(a.w, b.w);
                    }
                }
                x[k] = a;
            }
        }
        if (scale != 1.0f) {
#pragma unroll
            for (int k = 0; k < QMAX_V4; ++k) {
                x[k].x = __fmul_rn(x[k].x, scale); x[k].y = __fmul_rn(x[k].y, scale);
                x[k].z = __fmul_rn(x[k].z, scale); x[k].w = __fmul_rn(x[k].w, scale);
            }
        }
        if (proj_out) {
            float4* o = reinterpret_cast<float4*>(proj_out + row * d) + tid;
#pragma unroll
            for (int k = 0; k < QMAX_V4; ++k)
                if (FULL || tid + k * QT < nv4) __stcs(o + k * QT, x[k]);
        }
        // ---- one block reduction for both Eq. 2 and Eq. 4: sum of squares (double) and max |x| of the raw row.
        // yhat_m = fl(x_m * rn) is monotone in |x_m|, so max_m |yhat_m| = fl(max_m |x_m| * rn) exactly.
        double acc = 0.0;
        float mx = 0.0f;
        if (normalize) {
#pragma unroll
            for (int k = 0; k < QMAX_V4; ++k) {
                acc += (double)x[k].x * (double)x[k].x; acc += (double)x[k].y * (double)x[k].y;
                acc += (double)x[k].z * (double)x[k].z; acc += (double)x[k].w * (double)x[k].w;
            }
            acc = warp_sum(acc);
        }
#pragma unroll
        for (int k = 0; k < QMAX_V4; ++k)
            mx = fmaxf(fmaxf(mx, fmaxf(fabsf(x[k].x), fabsf(x[k].y))), fmaxf(fabsf(x[k].z), fabsf(x[k].w)));
        mx = warp_max(mx);
        if (lane == 0) { s_d[warp] = acc; s_f[warp] = mx; }
        __syncthreads();
        // One thread finishes the reduction and derives the row's scalars (the fp64 square root and the two IEEE
        // divisions are long instruction sequences: done by all 256 threads they were a tenth of the kernel's
        // instructions); the others pick them up behind a barrier.
        constexpr int ALPHA = (BITS == 1) ? 1 : ((1 << (BITS - 1)) - 1);
        if (tid == 0) {
            double tot = 0.0;
            float S0 = 0.0f;
#pragma unroll
            for (int w = 0; w < QT / 32; ++w) { tot += s_d[w]; S0 = fmaxf(S0, s_f[w]); }
            float rn0 = 1.0f;
            if (normalize) {
                const float nrm = (float)sqrt(tot);
                if (nrm == 0.0f) {
                    S0 = 0.0f;                              // zero vector
                } else {
                    rn0 = __fdiv_rn(1.0f, nrm);
                    S0 = __fmul_rn(S0, rn0);
                }
            }
            s_par[0] = rn0; s_par[1] = S0;
            s_par[2] = (S0 > 0.0f) ? __fdiv_rn((float)ALPHA, S0) : 0.0f;       // Eq. 5: alpha / S
        }
        __syncthreads();
        const float rn = s_par[0];
        float S = s_par[1], r = s_par[2];

        // ---- Eq. 5 + pack into shared memory ----
        if (ABSMEAN) {
            // gamma = mean |yhat| (sum in double), Delta = gamma * c_b (c_2 = 1, c_4 = 1/2, c_8 = 1/32),
            // q = clamp(rne(yhat / Delta), -alpha, alpha); the stored scale alpha * Delta dequantises like an absmax one
            double sa = 0.0;
#pragma unroll
            for (int k = 0; k < QMAX_V4; ++k) {
                sa += (double)fabsf(__fmul_rn(x[k].x, rn)); sa += (double)fabsf(__fmul_rn(x[k].y, rn));
                sa += (double)fabsf(__fmul_rn(x[k].z, rn)); sa += (double)fabsf(__fmul_rn(x[k].w, rn));
            }
            sa = warp_sum(sa);
            if (lane == 0) s_d[warp] = sa;       // s_d of the first reduction was read before the barrier above
            __syncthreads();
            if (tid == 0) {
                double ta = 0.0;
#pragma unroll
                for (int w = 0; w < QT / 32; ++w) ta += s_d[w];
                const float gamma = (float)(ta / (double)d);
                constexpr float CB = (BITS == 2) ? 1.0f : (BITS == 4) ? 0.5f : 0.03125f;
                const float delta = __fmul_rn(gamma, CB);
                s_par[2] = (gamma > 0.0f) ? __fdiv_rn(1.0f, delta) : 0.0f;
                s_par[1] = (gamma > 0.0f) ? __fmul_rn((float)ALPHA, delta) : 0.0f;
            }
            __syncthreads();
            S = s_par[1]; r = s_par[2];
        }
        int ss = 0;
#pragma unroll
        for (int k = 0; k < QMAX_V4; ++k) {
            const int c = tid + k * QT;
            if (FULL || c < nv4) {      // warp-uniform: nv4 is a multiple of 32
                const float e[4] = {__fmul_rn(x[k].x, rn), __fmul_rn(x[k].y, rn), __fmul_rn(x[k].z, rn), __fmul_rn(x[k].w, rn)};
                if (BITS == 1) {
                    uint32_t nib = 0;
#pragma unroll
                    for (int u = 0; u < 4; ++u) nib |= (e[u] < 0.0f) ? (1u << u) : 0u;     // a zero vector (S = 0) has no negative entry
                    const uint32_t hi = __shfl_down_sync(0xFFFFFFFFu, nib, 1);
                    if ((lane & 1) == 0) s_out[c >> 1] = (uint8_t)(nib | (hi << 4));
                } else {
                    // round-half-even to an integer by adding 1.5 * 2^23: the sum's low mantissa bits are the
                    // two's-complement code (|yhat r| <= alpha (1 + 2^-23), so no clamp is needed)
                    uint32_t t[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float v = __fmul_rn(e[u], r);
                        if (ABSMEAN) v = fminf(fmaxf(v, -(float)ALPHA), (float)ALPHA);      // clip (integers: rounding commutes)
                        t[u] = __float_as_uint(__fadd_rn(v, 12582912.0f));
                    }
                    // low bytes of the four sums -> one word of four int8 codes
                    const uint32_t w8 = __byte_perm(__byte_perm(t[0], t[1], 0x0040), __byte_perm(t[2], t[3], 0x0040), 0x5410);
                    ss = __dp4a((int)w8, (int)w8, ss);
                    if (BITS == 8) {
                        reinterpret_cast<uint32_t*>(s_out)[c] = w8;
                    } else if (BITS == 4) {
                        const uint32_t n4 = w8 & 0x0F0F0F0Fu;
                        const uint32_t u4 = n4 | (n4 >> 4);                    // bytes 0 and 2 hold two nibbles each
                        reinterpret_cast<uint16_t*>(s_out)[c] = (uint16_t)__byte_perm(u4, 0u, 0x4420);
                    } else {
                        const uint32_t n2 = w8 & 0x03030303u;
                        const uint32_t u2 = n2 | (n2 >> 6);                    // byte 0: codes 0,1 ; byte 2: codes 2,3
                        const uint32_t v2 = u2 | (u2 >> 12);                   // byte 0: codes 0..3
                        s_out[c] = (uint8_t)(v2 & 0xFFu);
                    }
                }
            }
        }
        if (BITS > 1) {
            ss = warp_sum_i(ss);
            if (lane == 0) s_i[warp] = ss;
        }
        __syncthreads();       // s_out and s_i complete
        if (tid == 0) {
            int tot = (S > 0.0f) ? d : 0;         // sign codes: every q^2 is 1, unless the vector is the zero vector
            if (BITS > 1) {
                tot = 0;
#pragma unroll
                for (int w = 0; w < QT / 32; ++w) tot += s_i[w];
            }
            scales[row] = S;
            if (sumsq) sumsq[row] = tot;
        }
        // ---- 128-bit coalesced stores of the packed row ----
        uint4* dst = reinterpret_cast<uint4*>(codes + row * (int64_t)row_bytes);
        const uint4* src = reinterpret_cast<const uint4*>(s_out);
        for (int i = tid; i < (row_bytes >> 4); i += QT) __stcs(dst + i, src[i]);
        __syncthreads();       // before the next row reuses shared memory
    }
}

}  // namespace

cudaError_t launch_quantize_absmean(const float* x, int64_t n, int32_t d, int normalize, int32_t bits, void* codes,
                                    float* scales, int32_t* sumsq, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    int64_t blocks = n;
    const int64_t cap = (int64_t)sm_count() * 8 * 4;
    if (blocks > cap) blocks = cap;
    uint8_t* c = reinterpret_cast<uint8_t*>(codes);
#define QLESS_QA(B, F) quantize_kernel<B, (B > 1), F><<<(unsigned)blocks, QT, 0, st>>>(x, 1, 1.0f, n, d, normalize, c, scales, sumsq, nullptr)
    const bool full = (d == QT * QMAX_V4 * 4);
    switch (bits) {
        case 8: if (full) QLESS_QA(8, true); else QLESS_QA(8, false); break;
        case 4: if (full) QLESS_QA(4, true); else QLESS_QA(4, false); break;
        case 2: if (full) QLESS_QA(2, true); else QLESS_QA(2, false); break;
        default: if (full) QLESS_QA(1, true); else QLESS_QA(1, false); break;
    }
#undef QLESS_QA
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_quantize(const float* parts, int32_t num_parts, float scale, int64_t n, int32_t d,
                            int normalize, int32_t bits, void* codes, float* scales, int32_t* sumsq,
                            float* proj_out, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    int64_t blocks = n;
    const int64_t cap = (int64_t)sm_count() * 8 * 4;
    if (blocks > cap) blocks = cap;
    uint8_t* c = reinterpret_cast<uint8_t*>(codes);
#define QLESS_Q(B, F, M) quantize_kernel<B, false, F, M><<<(unsigned)blocks, QT, 0, st>>>(parts, num_parts, scale, n, d, normalize, c, scales, sumsq, proj_out)
#define QLESS_QB(B) do { if (full && multi) QLESS_Q(B, true, true); else if (full) QLESS_Q(B, true, false); \
                         else if (multi) QLESS_Q(B, false, true); else QLESS_Q(B, false, false); } while (0)
    const bool full = (d == QT * QMAX_V4 * 4), multi = (num_parts > 1);
    switch (bits) {
        case 8: QLESS_QB(8); break;
        case 4: QLESS_QB(4); break;
        case 2: QLESS_QB(2); break;
        default: QLESS_QB(1); break;
    }
#undef QLESS_QB
#undef QLESS_Q
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace qless
