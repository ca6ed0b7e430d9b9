// Stage 3 on the CUDA cores: integer similarity (XOR + POPC for 1-bit codes, 4-way int8 dot
// instructions for 8/4/2-bit codes unpacked in shared memory), followed in the same kernel by the
// per-vector multipliers, the per-task mean, the learning-rate-weighted sum over checkpoints and
// the max over tasks (Eq. 6-7 and the LESS aggregation).
#include "qless_kernels.h"

namespace qless {

namespace {

constexpr int TT = 64;        // train rows per CTA
constexpr int TV = 128;       // validation rows per tile
constexpr int KW = 64;        // operand words per K-chunk
constexpr int LDW = KW + 4;   // padded row length in words (16-byte rows, conflict-free 128-bit reads)
constexpr int ST = 256;

// Copies one K-chunk of `rows` code rows into shared memory as operand words.
// BITS = 1: words are the packed sign words. BITS > 1: each word holds four sign-extended int8 codes;
// the order of codes inside a chunk is a fixed permutation, identical for both operands.
template <int BITS>
__device__ __forceinline__ void load_chunk(uint32_t* __restrict__ dst, const uint8_t* __restrict__ src,
                                           int64_t row0, int64_t row_end, int rows, int row_bytes, int kc)
{
    constexpr int OUT_PER_SRC = (BITS == 1) ? 1 : 8 / BITS;
    constexpr int SRC_WORDS = KW / OUT_PER_SRC;                 // source words per row per chunk
    const int src_word0 = kc / OUT_PER_SRC;
    const int row_src_words = row_bytes >> 2;
    for (int e = threadIdx.x; e < rows * SRC_WORDS; e += ST) {
        const int row = e / SRC_WORDS, sw = e - row * SRC_WORDS;
        uint32_t w = 0;
        const bool ok = (row0 + row < row_end) && (src_word0 + sw < row_src_words);
        if (ok) w = __ldg(reinterpret_cast<const uint32_t*>(src + (row0 + row) * (int64_t)row_bytes) + src_word0 + sw);
        uint32_t* o = dst + row * LDW + sw * OUT_PER_SRC;
        if (BITS == 1 || BITS == 8) {
            o[0] = w;
        } else if (BITS == 4) {
            o[0] = __vsub4((w & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);
            o[1] = __vsub4(((w >> 4) & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);
        } else {
#pragma unroll
            for (int f = 0; f < 4; ++f)
                o[f] = __vsub4(((w >> (2 * f)) & 0x03030303u) ^ 0x02020202u, 0x02020202u);
        }
    }
}

template <int BITS>
__global__ void __launch_bounds__(ST)
score_simt_kernel(ScoreArgs a)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    uint32_t* s_train = reinterpret_cast<uint32_t*>(smem_raw);          // [TT][LDW]
    uint32_t* s_val = s_train + TT * LDW;                                // [TV][LDW]
    float* s_sim = reinterpret_cast<float*>(s_val + TV * LDW);           // [TT][TV+1]
    float* s_A = s_sim + TT * (TV + 1);                                  // [TT][T]

    const int tid = threadIdx.x;
    const int ty = tid >> 4, tx = tid & 15;       // thread tile: train rows ty + 16*u (u<4), val rows tx + 16*w (w<8)
    const int row_bytes = a.d * BITS / 8;
    const int words_per_row = (BITS == 1) ? a.d / 32 : a.d / 4;
    const int64_t t0 = (int64_t)blockIdx.x * TT;

    for (int e = tid; e < TT * a.T; e += ST) s_A[e] = 0.0f;

    for (int i = 0; i < a.C; ++i) {
        const uint8_t* tr = a.train + i * a.train_stride;
        const uint8_t* va = a.val + i * a.val_stride;
        for (int v0 = 0; v0 < a.V; v0 += TV) {
            int acc[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int w = 0; w < 8; ++w) acc[u][w] = 0;

            for (int kc = 0; kc < words_per_row; kc += KW) {
                __syncthreads();
                load_chunk<BITS>(s_train, tr, t0, a.N, TT, row_bytes, kc);
                load_chunk<BITS>(s_val, va, v0, a.V, TV, row_bytes, kc);
                __syncthreads();
#pragma unroll 4
                for (int k4 = 0; k4 < KW; k4 += 4) {
                    uint4 x[4], y[8];
#pragma unroll
                    for (int u = 0; u < 4; ++u) x[u] = *reinterpret_cast<const uint4*>(s_train + (ty + 16 * u) * LDW + k4);
#pragma unroll
                    for (int w = 0; w < 8; ++w) y[w] = *reinterpret_cast<const uint4*>(s_val + (tx + 16 * w) * LDW + k4);
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int w = 0; w < 8; ++w) {
                            if (BITS == 1) {
                                acc[u][w] += __popc(x[u].x ^ y[w].x) + __popc(x[u].y ^ y[w].y) +
                                             __popc(x[u].z ^ y[w].z) + __popc(x[u].w ^ y[w].w);
                            } else {
                                int s = acc[u][w];
                                s = __dp4a((int)x[u].x, (int)y[w].x, s);
                                s = __dp4a((int)x[u].y, (int)y[w].y, s);
                                s = __dp4a((int)x[u].z, (int)y[w].z, s);
                                s = __dp4a((int)x[u].w, (int)y[w].w, s);
                                acc[u][w] = s;
                            }
                        }
                }
            }
            // ---- epilogue of this (checkpoint, validation tile) ----
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int w = 0; w < 8; ++w) {
                    const int D = (BITS == 1) ? (a.d - 2 * acc[u][w]) : acc[u][w];
                    const int tl = ty + 16 * u, vl = tx + 16 * w;
                    const int64_t t = t0 + tl;
                    const int v = v0 + vl;
                    if (a.dots) {
                        if (i == 0 && t < a.N && v < a.V) a.dots[t * a.V + v] = D;
                    } else {
                        const float mv = (v < a.V) ? a.val_mult[(int64_t)i * a.V + v] : 0.0f;
                        s_sim[tl * (TV + 1) + vl] = __fmul_rn((float)D, mv);
                    }
                }
            if (!a.dots) {
                __syncthreads();
                for (int e = tid; e < TT * a.T; e += ST) {
                    const int tl = e / a.T, j = e - tl * a.T;
                    const int64_t t = t0 + tl;
                    const int lo = max(a.task_off[j], v0), hi = min(a.task_off[j + 1], v0 + TV);
                    if (t < a.N && lo < hi) {
                        float s = 0.0f;
                        for (int v = lo; v < hi; ++v) s += s_sim[tl * (TV + 1) + (v - v0)];
                        const float mt = a.train_mult[(int64_t)i * a.N + t];
                        s_A[e] += s * mt * a.eta_over_cnt[i * a.T + j];
                    }
                }
            }
        }
        if (a.dots) break;     // raw dots: one checkpoint only
    }
    if (a.dots) return;
    __syncthreads();
    for (int tl = tid; tl < TT; tl += ST) {
        const int64_t t = t0 + tl;
        if (t < a.N) {
            float best = s_A[tl * a.T];
            for (int j = 1; j < a.T; ++j) best = fmaxf(best, s_A[tl * a.T + j]);
            a.scores[t] = best;
        }
    }
    if (a.per_task)
        for (int e = tid; e < TT * a.T; e += ST) {
            const int tl = e / a.T;
            if (t0 + tl < a.N) a.per_task[t0 * a.T + e] = s_A[e];
        }
}

// mult = 0 for a zero vector (scale == 0); cosine: 1/sqrt(||q||^2); dequant: scale/alpha.
template <int BITS>
__global__ void multipliers_kernel(const uint8_t* __restrict__ codes, int64_t ckpt_stride,
                                   const float* __restrict__ scales, const int32_t* __restrict__ sumsq,
                                   int64_t rows, int32_t C, int32_t d, int mode, float* __restrict__ mult)
{
    // one warp per vector
    const int lane = threadIdx.x & 31;
    const int64_t vec = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (vec >= rows * C) return;
    const int64_t i = vec / rows, t = vec - i * rows;
    const float S = scales[vec];
    float m = 0.0f;
    if (S != 0.0f) {
        if (mode == 1) {
            constexpr int ALPHA = (BITS == 1) ? 1 : ((1 << (BITS - 1)) - 1);
            m = __fdiv_rn(S, (float)ALPHA);
        } else {
            int ss;
            if (sumsq) {
                ss = sumsq[vec];
            } else if (BITS == 1) {
                ss = d;
            } else {
                const int row_bytes = d * BITS / 8;
                const uint32_t* p = reinterpret_cast<const uint32_t*>(codes + i * ckpt_stride + t * (int64_t)row_bytes);
                int acc = 0;
                for (int w = lane; w < (row_bytes >> 2); w += 32) {
                    const uint32_t x = p[w];
                    if (BITS == 8) {
                        acc = __dp4a((int)x, (int)x, acc);
                    } else if (BITS == 4) {
                        const uint32_t lo = __vsub4((x & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);
                        const uint32_t hi = __vsub4(((x >> 4) & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);
                        acc = __dp4a((int)lo, (int)lo, acc);
                        acc = __dp4a((int)hi, (int)hi, acc);
                    } else {
#pragma unroll
                        for (int f = 0; f < 4; ++f) {
                            const uint32_t y = __vsub4(((x >> (2 * f)) & 0x03030303u) ^ 0x02020202u, 0x02020202u);
                            acc = __dp4a((int)y, (int)y, acc);
                        }
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                ss = acc;
            }
            m = (ss > 0) ? (float)(1.0 / sqrt((double)ss)) : 0.0f;
        }
    }
    if (lane == 0) mult[vec] = m;
}

size_t score_smem_bytes(int T) { return (size_t)(TT + TV) * LDW * 4 + (size_t)TT * (TV + 1) * 4 + (size_t)TT * T * 4; }

}  // namespace

cudaError_t launch_score_simt(const ScoreArgs& a, cudaStream_t st)
{
    if (a.N == 0) return cudaSuccess;
    const size_t smem = score_smem_bytes(a.T);
    const unsigned grid = (unsigned)((a.N + TT - 1) / TT);
    cudaError_t e;
#define QLESS_LAUNCH_SCORE(B)                                                                               \
    e = cudaFuncSetAttribute(score_simt_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                                         \
    score_simt_kernel<B><<<grid, ST, smem, st>>>(a);
    switch (a.bits) {
        case 8: QLESS_LAUNCH_SCORE(8) break;
        case 4: QLESS_LAUNCH_SCORE(4) break;
        case 2: QLESS_LAUNCH_SCORE(2) break;
        default: QLESS_LAUNCH_SCORE(1) break;
    }
#undef QLESS_LAUNCH_SCORE
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_multipliers(const uint8_t* codes, int64_t ckpt_stride, const float* scales,
                               const int32_t* sumsq, int64_t rows, int32_t C, int32_t d, int32_t bits, int mode,
                               float* mult, cudaStream_t st)
{
    const int64_t vecs = rows * C;
    if (vecs == 0) return cudaSuccess;
    const unsigned grid = (unsigned)((vecs * 32 + 255) / 256);
    switch (bits) {
        case 8: multipliers_kernel<8><<<grid, 256, 0, st>>>(codes, ckpt_stride, scales, sumsq, rows, C, d, mode, mult); break;
        case 4: multipliers_kernel<4><<<grid, 256, 0, st>>>(codes, ckpt_stride, scales, sumsq, rows, C, d, mode, mult); break;
        case 2: multipliers_kernel<2><<<grid, 256, 0, st>>>(codes, ckpt_stride, scales, sumsq, rows, C, d, mode, mult); break;
        default: multipliers_kernel<1><<<grid, 256, 0, st>>>(codes, ckpt_stride, scales, sumsq, rows, C, d, mode, mult); break;
    }
    count_launches(1);
    return cudaGetLastError();
}

// 16-bit baseline: mult[i][r] = 1 / ||row r of checkpoint i|| (0 for a zero row), rows of d bf16 values. One warp per
// row, squares summed in double.
__global__ void __launch_bounds__(256)
inv_norm_bf16_kernel(const uint8_t* __restrict__ rows, int64_t ckpt_stride, int64_t nrows, int32_t C, int32_t d,
                     float* __restrict__ mult)
{
    const int lane = threadIdx.x & 31;
    const int64_t nwarp = (int64_t)gridDim.x * 8;
    for (int64_t r = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); r < (int64_t)C * nrows; r += nwarp) {
        const int64_t i = r / nrows, row = r - i * nrows;
        const uint4* src = reinterpret_cast<const uint4*>(rows + i * ckpt_stride + row * (int64_t)d * 2);
        double acc = 0.0;
        for (int c = lane; c < d / 8; c += 32) {
            const uint4 w = __ldg(src + c);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const double lo = (double)__uint_as_float(ww[u] << 16), hi = (double)__uint_as_float(ww[u] & 0xFFFF0000u);
                acc += lo * lo; acc += hi * hi;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) mult[r] = (acc > 0.0) ? (float)(1.0 / sqrt(acc)) : 0.0f;
    }
}

cudaError_t launch_inv_norms_bf16(const uint8_t* rows, int64_t ckpt_stride, int64_t nrows, int32_t C, int32_t d,
                                  float* mult, cudaStream_t st)
{
    if (nrows == 0) return cudaSuccess;
    int64_t blocks = ((int64_t)C * nrows + 7) / 8;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    inv_norm_bf16_kernel<<<(unsigned)blocks, 256, 0, st>>>(rows, ckpt_stride, nrows, C, d, mult);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace qless
