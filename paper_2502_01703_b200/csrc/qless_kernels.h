// Internal launch interface between the C ABI (api.cu) and the kernel translation units.
#pragma once
#include <cuda.h>

#include "qless_common.cuh"

namespace qless {

struct AdamParams {
    float beta1, beta2, eps;
    float omb1, omb2;      // 1 - beta1, 1 - beta2 (fp32 subtraction, as written in the formula)
    float c1, c2;          // bias-correction divisors (1 if step == 0)
    int   bias_correct;
};

// Gamma (bf16) from gradient rows; m/v NULL => bf16(g). tiled = false: row-major [n, P];
// tiled = true: [P/64][n][64] (element (i, j) at ((j/64)*n + i)*64 + j%64), the layout the projection reads.
cudaError_t launch_adam_gamma(const void* grads, qless_dtype dtype, int64_t n, int64_t ld,
                              const float* m, const float* v, const AdamParams& ap, int64_t P,
                              __nv_bfloat16* gamma, bool tiled, cudaStream_t st);

cudaError_t launch_philox_entries(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj,
                                  int8_t* out, cudaStream_t st);
// Entries of the Gaussian matrix as fp32 (bf16-representable values); j0 a multiple of 4.
cudaError_t launch_gaussian_entries(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj,
                                    float* out, cudaStream_t st);

// Projection partial sums: part[s][i][r] = sum over K-chunk s of Gamma[i][j] * sign(r, j), fp32,
// s = 0 .. num_chunks-1, chunk s covering columns [s*chunk, min(P, (s+1)*chunk)).
struct ProjectPlan {
    int64_t n, P;
    int32_t d;
    int64_t chunk;        // K-chunk length (multiple of 128)
    int32_t num_chunks;
    int64_t k_base;       // absolute index of the first column given (a multiple of chunk): offsets the Philox counters
    bool gaussian;        // entries of R: false = Rademacher +-1 (the method), true = standard normal (bf16)
};
ProjectPlan plan_projection(int64_t n, int64_t P, int32_t d);
cudaError_t launch_project_simt(const __nv_bfloat16* gamma_tiled, const ProjectPlan& pl,
                                uint64_t seed, float* part, cudaStream_t st);

// Tensor-core projection (project_tc.cu). The tensor map describes tiled Gamma as [(P/64)*n][64] bf16 with a
// 64 x 128 box.
cudaError_t launch_project_tc(const CUtensorMap& tmap, const ProjectPlan& pl, uint64_t seed, float* part,
                              unsigned int* timeout_word, cudaStream_t st);

// Stage 2. x = inv_scale-scaled sum of `num_parts` partial arrays [num_parts][n][d] (num_parts = 1,
// scale = 1 for plain rows). Writes proj_out (optional), codes, scales, sumsq (optional).
// Absmean variant of the same stage on plain fp32 rows (scale from the mean absolute value).
cudaError_t launch_quantize_absmean(const float* x, int64_t n, int32_t d, int normalize, int32_t bits, void* codes,
                                    float* scales, int32_t* sumsq, cudaStream_t st);
cudaError_t launch_quantize(const float* parts, int32_t num_parts, float scale, int64_t n, int32_t d,
                            int normalize, int32_t bits, void* codes, float* scales, int32_t* sumsq,
                            float* proj_out, cudaStream_t st);

// Stage 3.
struct ScoreArgs {
    const uint8_t* train; int64_t train_stride;   // bytes per checkpoint
    const uint8_t* val;   int64_t val_stride;
    const float* train_mult;    // [C][N] per-vector multipliers
    const float* val_mult;      // [C][V]
    const float* eta_over_cnt;  // device [C][T]: eta_i / |task j|
    const int32_t* task_off;    // device [T+1]
    int64_t N; int32_t V, C, T, d, bits;
    float* scores; float* per_task;
    int32_t* dots;              // if non-NULL: write raw integer dots [N][V] of checkpoint 0 only
};
cudaError_t launch_score_simt(const ScoreArgs& a, cudaStream_t st);
// Tensor-core scoring (score_tc.cu) for bits in {8, 4, 2, 1}, and for bits = 16: rows of d bf16 values, fp32
// accumulation (the 16-bit baseline). T must be <= 8 (score_tc_supported).
bool score_tc_supported(int32_t T);
size_t score_tc_workspace_bytes(int32_t V, int32_t C, int32_t d, int32_t bits);
qless_status launch_score_tc(const ScoreArgs& a, uint8_t* val_unpacked, unsigned int* timeout_word, cudaStream_t st);
// multipliers: mult = (scale == 0) ? 0 : 1/sqrt(sumsq) (cosine) or scale/alpha (dequant);
// sumsq NULL => recomputed from codes.
cudaError_t launch_multipliers(const uint8_t* codes, int64_t ckpt_stride, const float* scales,
                               const int32_t* sumsq, int64_t rows, int32_t C, int32_t d, int32_t bits,
                               int mode, float* mult, cudaStream_t st);
// 16-bit baseline: per-row 1/norm of bf16 rows [C][nrows][d] (0 for a zero row).
cudaError_t launch_inv_norms_bf16(const uint8_t* rows, int64_t ckpt_stride, int64_t nrows, int32_t C, int32_t d,
                                  float* mult, cudaStream_t st);

// Stage 4.
size_t select_workspace_bytes(int64_t N);
cudaError_t launch_select_topk(const float* scores, int64_t N, int64_t k, int64_t* indices,
                               void* ws, cudaStream_t st);
// 0: path by size; 1: multi-pass select at every N; 2: sampled bracket forced too high (exercises the fallback).
void set_select_path(int mode);

}  // namespace qless
