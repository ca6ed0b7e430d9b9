// Shared host/device helpers of the QLESS CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "qless.h"

namespace qless {

// ---- error plumbing --------------------------------------------------------------------------
qless_status fail(qless_status st, const char* fmt, ...);   // records the thread-local message
qless_status cuda_fail(cudaError_t e, const char* what);

#define QLESS_CUDA_TRY(expr)                                              \
    do {                                                                  \
        cudaError_t e__ = (expr);                                         \
        if (e__ != cudaSuccess) return ::qless::cuda_fail(e__, #expr);    \
    } while (0)

#define QLESS_REQUIRE(cond, st, ...)                                      \
    do {                                                                  \
        if (!(cond)) return ::qless::fail((st), __VA_ARGS__);             \
    } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Optional per-kernel event timing (see qless_profile_enable). Usage: { ProfileScope ps("name", st); launch; }
struct ProfileScope {
    ProfileScope(const char* name, cudaStream_t st);
    ~ProfileScope();
    const char* name_; cudaStream_t st_; int slot_;
};

void count_launches(int n);   // bookkeeping behind qless_kernel_launches()

int sm_count();   // SM count of the current device (cached)

// Address of the device-side timeout word that kernels with bounded waits set when they give up.
unsigned int* timeout_flag_ptr();

// ---- Philox4x32-10 (Salmon et al., SC'11) ----------------------------------------------------
__host__ __device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                       uint32_t k0, uint32_t k1, uint32_t (&out)[4])
{
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
#ifdef __CUDA_ARCH__
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
#else
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
#endif
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Random words of the 128 matrix entries (row r, columns 128*blk .. 128*blk+127).
__device__ __forceinline__ void rademacher_block(uint64_t seed, uint32_t r, uint32_t blk, uint32_t (&w)[4])
{
    philox4x32_10(blk, r, 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), w);
}

// Two consecutive entries (columns 2p, 2p+1 of a 32-column group; p = 0..15) of a random word as
// a packed bf16 pair {+-1.0, +-1.0}: column 2p takes bit 15-p, column 2p+1 takes bit 31-p, so one
// left shift lines both up with the bf16 sign bits.
__device__ __forceinline__ uint32_t rademacher_bf16x2(uint32_t word, int p)
{
    return ((word << p) & 0x80008000u) | 0x3F803F80u;
}

// Sign (+1/-1) of entry u = 0..31 of a random word.
__host__ __device__ __forceinline__ int rademacher_sign_of(uint32_t word, int u)
{
    const int beta = 15 - (u >> 1) + 16 * (u & 1);
    return ((word >> beta) & 1u) ? -1 : 1;
}

// Gaussian matrix (the other distribution Sec. 2.4 allows): the four entries of row r in columns 4q .. 4q+3 come
// from one Philox call with counter (q mod 2^32, r, q div 2^32, 1); output words (w0, w1) give columns 4q, 4q+1 and
// (w2, w3) give 4q+2, 4q+3 by the Box-Muller transform of u = (floor(w / 2^9) + 1/2) / 2^23 (exact in fp32,
// strictly inside (0, 1)): z_even = sqrt(-2 ln u1) cos(2 pi u2), z_odd = sqrt(-2 ln u1) sin(2 pi u2). The entries
// are rounded to bf16, the operand type of the contraction; lo packs columns 4q, 4q+1 (4q in the low half),
// hi packs 4q+2, 4q+3.
#ifdef __CUDACC__
__device__ __forceinline__ uint32_t box_muller_bf16x2(uint32_t wa, uint32_t wb)
{
    // The generator warps bound this variant, so the transform runs on the special-function units: log2, square
    // root, sine and cosine each one approximate instruction (absolute error about 2^-21 with the angle brought
    // into (-pi, pi): cos(2 pi u2) = -cos(2 pi (u2 - 1/2)), likewise the sine), well inside half a bf16 step except
    // for entries that sit next to a rounding boundary.
    const float u1 = ((float)(wa >> 9) + 0.5f) * 1.1920928955078125e-07f;                 // 2^-23, exact
    const float t = ((float)((int)(wb >> 9) - (1 << 22)) + 0.5f) * 1.1920928955078125e-07f;   // u2 - 1/2, exact
    float rho;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rho) : "f"(-2.0f * __logf(u1)));
    const float ang = 6.283185307179586f * t;
    const __nv_bfloat162 z = __floats2bfloat162_rn(-rho * __cosf(ang), -rho * __sinf(ang));
    return *reinterpret_cast<const uint32_t*>(&z);
}
__device__ __forceinline__ void gaussian_quad_bf16x2(uint64_t seed, uint32_t r, uint32_t q_lo, uint32_t q_hi,
                                                     uint32_t& lo, uint32_t& hi)
{
    uint32_t w[4];
    philox4x32_10(q_lo, r, q_hi, 1u, (uint32_t)seed, (uint32_t)(seed >> 32), w);
    lo = box_muller_bf16x2(w[0], w[1]);
    hi = box_muller_bf16x2(w[2], w[3]);
}
#endif

// Order-preserving key of an fp32 score: larger key <=> larger score; -0 < +0; NaN lowest.
__host__ __device__ __forceinline__ uint32_t order_key(uint32_t bits)
{
    if ((bits & 0x7F800000u) == 0x7F800000u && (bits & 0x007FFFFFu)) return 0u;
    return (bits >> 31) ? ~bits : (bits | 0x80000000u);
}

}  // namespace qless
