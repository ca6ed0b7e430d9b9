// C ABI of the QLESS library: argument validation, workspace carving and kernel sequencing.
#include <mutex>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <vector>

#include "qless_kernels.h"
#include "tc_common.cuh"

namespace qless {

static thread_local char t_err[512] = "";

qless_status fail(qless_status st, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_err, sizeof(t_err), fmt, ap);
    va_end(ap);
    return st;
}

qless_status cuda_fail(cudaError_t e, const char* what)
{
    snprintf(t_err, sizeof(t_err), "CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
    return QLESS_ERR_CUDA;
}

static std::atomic<uint64_t> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int sm_count()
{
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached = n; cached_dev = dev;
    }
    return cached;
}

__device__ unsigned int g_timeout_flag = 0;

unsigned int* timeout_flag_ptr()
{
    static thread_local int cached_dev = -1;
    static thread_local unsigned int* p = nullptr;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev != cached_dev || p == nullptr) {
        void* q = nullptr;
        if (cudaGetSymbolAddress(&q, g_timeout_flag) != cudaSuccess) return nullptr;
        p = reinterpret_cast<unsigned int*>(q); cached_dev = dev;
    }
    return p;
}

// ---- per-kernel event timing ---------------------------------------------------------------------
struct ProfRec { const char* name; cudaEvent_t a, b; };
static thread_local bool t_prof_on = false;
static thread_local std::vector<ProfRec> t_prof;

ProfileScope::ProfileScope(const char* name, cudaStream_t st) : name_(name), st_(st), slot_(-1)
{
    if (!t_prof_on) return;
    ProfRec r; r.name = name;
    if (cudaEventCreate(&r.a) != cudaSuccess) return;
    if (cudaEventCreate(&r.b) != cudaSuccess) { cudaEventDestroy(r.a); return; }
    cudaEventRecord(r.a, st);
    t_prof.push_back(r);
    slot_ = (int)t_prof.size() - 1;
}
ProfileScope::~ProfileScope()
{
    if (slot_ >= 0) cudaEventRecord(t_prof[slot_].b, st_);
}

static std::atomic<int> g_score_path{0};        // 0 = tensor cores for 8/4/2-bit codes, 1 = CUDA cores
static std::atomic<int> g_projection_path{0};   // 0 = tensor cores, 1 = CUDA cores (cross-check hook)

static bool valid_bits(int b) { return b == 1 || b == 2 || b == 4 || b == 8; }
static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static qless_status make_adam(const qless_adam_cfg* cfg, AdamParams* ap)
{
    qless_adam_cfg c = {0.9f, 0.999f, 1e-8f, 0};
    if (cfg) c = *cfg;
    QLESS_REQUIRE(c.beta1 >= 0.f && c.beta1 < 1.f && c.beta2 >= 0.f && c.beta2 < 1.f && c.eps >= 0.f && c.step >= 0,
                  QLESS_ERR_INVALID_ARG, "adam config out of range (beta in [0,1), eps >= 0, step >= 0)");
    ap->beta1 = c.beta1; ap->beta2 = c.beta2; ap->eps = c.eps;
    ap->omb1 = 1.0f - c.beta1; ap->omb2 = 1.0f - c.beta2;
    ap->bias_correct = c.step > 0;
    ap->c1 = ap->c2 = 1.0f;
    if (c.step > 0) {
        ap->c1 = (float)(1.0 - std::pow((double)c.beta1, (double)c.step));
        ap->c2 = (float)(1.0 - std::pow((double)c.beta2, (double)c.step));
    }
    return QLESS_OK;
}

// The random matrix of Eq. 1 travels with the call: NULL = Rademacher.
static qless_status matrix_kind(const qless_projection_cfg* cfg, bool* gaussian)
{
    *gaussian = false;
    if (cfg == nullptr) return QLESS_OK;
    QLESS_REQUIRE(cfg->matrix == QLESS_MATRIX_RADEMACHER || cfg->matrix == QLESS_MATRIX_GAUSSIAN, QLESS_ERR_INVALID_ARG,
                  "projection->matrix must be QLESS_MATRIX_RADEMACHER (0) or QLESS_MATRIX_GAUSSIAN (1) (matrix=%d)", cfg->matrix);
    QLESS_REQUIRE(cfg->reserved[0] == 0 && cfg->reserved[1] == 0 && cfg->reserved[2] == 0, QLESS_ERR_INVALID_ARG,
                  "projection->reserved must be zero");
    *gaussian = cfg->matrix == QLESS_MATRIX_GAUSSIAN;
    return QLESS_OK;
}

static qless_status check_grads(const void* grads, qless_dtype dtype, int64_t n, int64_t ld, const float* m,
                                const float* v, int64_t P)
{
    QLESS_REQUIRE(n >= 0 && P > 0, QLESS_ERR_INVALID_ARG, "n must be >= 0 and P > 0 (n=%lld, P=%lld)", (long long)n, (long long)P);
    QLESS_REQUIRE(dtype == QLESS_F32 || dtype == QLESS_BF16, QLESS_ERR_INVALID_ARG, "dtype must be QLESS_F32 or QLESS_BF16");
    QLESS_REQUIRE(P % 128 == 0, QLESS_ERR_UNSUPPORTED, "P must be a multiple of 128 (P=%lld)", (long long)P);
    QLESS_REQUIRE(P < ((int64_t)1 << 39), QLESS_ERR_UNSUPPORTED, "P must be < 2^39");
    QLESS_REQUIRE((m == nullptr) == (v == nullptr), QLESS_ERR_INVALID_ARG, "adam_m and adam_v must both be given or both be NULL");
    if (n == 0) return QLESS_OK;
    QLESS_REQUIRE(grads != nullptr, QLESS_ERR_INVALID_ARG, "grads is NULL");
    QLESS_REQUIRE(ld >= P && ld % 8 == 0, QLESS_ERR_INVALID_ARG, "ld_grads must be >= P and a multiple of 8 (ld=%lld)", (long long)ld);
    QLESS_REQUIRE(aligned(grads, 16) && aligned(m, 16) && aligned(v, 16), QLESS_ERR_INVALID_ARG, "grads, adam_m, adam_v must be 16-byte aligned");
    return QLESS_OK;
}

struct PqWorkspace {
    size_t gamma_off, part_off, total;
    ProjectPlan plan;
};

static PqWorkspace pq_layout(int64_t n, int64_t P, int32_t d)
{
    PqWorkspace w;
    w.plan = plan_projection(n, P, d);
    w.gamma_off = 0;
    w.part_off = align_up((size_t)n * (size_t)P * sizeof(__nv_bfloat16), 256);
    w.total = w.part_off + align_up((size_t)w.plan.num_chunks * (size_t)n * (size_t)d * sizeof(float), 256);
    return w;
}

// Adam prologue and projection of the columns [j0, j0 + len) of a batch whose full plan is `full` (j0 and len
// multiples of full.chunk, except that the last range may end at P): Gamma goes to its place in the K-blocked
// buffer [P/64][n][64], the partial sums to the chunks of that range. Everything is enqueued on st.
static qless_status project_columns(const void* grads, qless_dtype dtype, int64_t n, int64_t ld_grads, const float* adam_m,
                                    const float* adam_v, const AdamParams& ap, const ProjectPlan& full, int64_t j0,
                                    int64_t len, uint64_t seed, bool gaussian, __nv_bfloat16* gamma, float* part,
                                    cudaStream_t st)
{
    const size_t esz = (dtype == QLESS_BF16) ? 2 : 4;
    const void* g_slab = reinterpret_cast<const uint8_t*>(grads) + (size_t)j0 * esz;
    __nv_bfloat16* gamma_slab = gamma + (j0 / 64) * n * 64;
    // Pre-pass: Gamma as bf16 in the K-blocked layout the projection streams
    { ProfileScope ps("adam_gamma", st);
      QLESS_CUDA_TRY(launch_adam_gamma(g_slab, dtype, n, ld_grads, adam_m ? adam_m + j0 : nullptr, adam_v ? adam_v + j0 : nullptr,
                                       ap, len, gamma_slab, true, st)); }
    ProjectPlan pl = full;
    pl.P = len; pl.k_base = j0;
    pl.gaussian = gaussian;
    pl.num_chunks = (int32_t)((len + full.chunk - 1) / full.chunk);
    float* part_slab = part + (j0 / full.chunk) * n * (int64_t)full.d;
    if (g_projection_path == 0 && (len / 64) * n < ((int64_t)1 << 31)) {
        CUtensorMap tmap;
        qless_status s = make_tmap_2d_sw128(&tmap, gamma_slab, 2, 64, (uint64_t)(len / 64) * (uint64_t)n, 128, 64, 128);
        if (s != QLESS_OK) return s;
        unsigned int* flag = timeout_flag_ptr();
        QLESS_REQUIRE(flag != nullptr, QLESS_ERR_CUDA, "cannot resolve the device timeout flag");
        ProfileScope ps("project", st);
        QLESS_CUDA_TRY(launch_project_tc(tmap, pl, seed, part_slab, flag, st));
    } else {
        ProfileScope ps("project", st);
        QLESS_CUDA_TRY(launch_project_simt(gamma_slab, pl, seed, part_slab, st));
    }
    return QLESS_OK;
}

// A stream of the library's own per device, for copies that run beside the caller's stream.
static qless_status copy_stream(cudaStream_t* out)
{
    static std::mutex mu;
    static cudaStream_t streams[64] = {};
    int dev = 0;
    QLESS_CUDA_TRY(cudaGetDevice(&dev));
    QLESS_REQUIRE(dev >= 0 && dev < 64, QLESS_ERR_UNSUPPORTED, "device ordinal %d beyond 64", dev);
    std::lock_guard<std::mutex> lk(mu);
    if (streams[dev] == nullptr) QLESS_CUDA_TRY(cudaStreamCreateWithFlags(&streams[dev], cudaStreamNonBlocking));
    *out = streams[dev];
    return QLESS_OK;
}

}  // namespace qless

using namespace qless;

extern "C" {

const char* qless_last_error(void) { return t_err; }

qless_status qless_check(void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    unsigned int* flag = timeout_flag_ptr();
    QLESS_REQUIRE(flag != nullptr, QLESS_ERR_CUDA, "cannot resolve the device timeout flag");
    unsigned int h = 0;
    QLESS_CUDA_TRY(cudaMemcpyAsync(&h, flag, sizeof(h), cudaMemcpyDeviceToHost, st));
    QLESS_CUDA_TRY(cudaStreamSynchronize(st));
    if (h != 0) {
        QLESS_CUDA_TRY(cudaMemsetAsync(flag, 0, sizeof(h), st));
        QLESS_CUDA_TRY(cudaStreamSynchronize(st));
        return fail(QLESS_ERR_TIMEOUT, "a device-side bounded wait gave up (code 0x%x); results of that call are invalid", h);
    }
    return QLESS_OK;
}

qless_status qless_set_projection_path(int32_t path)
{
    QLESS_REQUIRE(path == 0 || path == 1, QLESS_ERR_INVALID_ARG, "path must be 0 (tensor cores) or 1 (CUDA cores)");
    g_projection_path.store(path);
    return QLESS_OK;
}

qless_status qless_gaussian_entries(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj, float* out,
                                    void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(r0 >= 0 && nr >= 0 && j0 >= 0 && nj >= 0, QLESS_ERR_INVALID_ARG, "negative range");
    QLESS_REQUIRE(j0 % 4 == 0, QLESS_ERR_INVALID_ARG, "j0 must be a multiple of 4 (j0=%lld)", (long long)j0);
    QLESS_REQUIRE(r0 + nr <= ((int64_t)1 << 32) && j0 + nj <= ((int64_t)1 << 39), QLESS_ERR_UNSUPPORTED, "row < 2^32 and column < 2^39 required");
    if (nr == 0 || nj == 0) return QLESS_OK;
    QLESS_REQUIRE(out != nullptr, QLESS_ERR_INVALID_ARG, "out is NULL");
    QLESS_CUDA_TRY(launch_gaussian_entries(seed, r0, nr, j0, nj, out, st));
    return QLESS_OK;
}

qless_status qless_set_score_path(int32_t path)
{
    QLESS_REQUIRE(path == 0 || path == 1, QLESS_ERR_INVALID_ARG, "path must be 0 (tensor cores) or 1 (CUDA cores)");
    g_score_path.store(path);
    return QLESS_OK;
}

qless_status qless_set_select_path(int32_t path)
{
    QLESS_REQUIRE(path >= 0 && path <= 2, QLESS_ERR_INVALID_ARG, "path must be 0 (by size), 1 (multi-pass) or 2 (bracket forced too high)");
    set_select_path(path);
    return QLESS_OK;
}

uint64_t qless_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

qless_status qless_profile_enable(int32_t on)
{
    t_prof_on = on != 0;
    return QLESS_OK;
}

qless_status qless_profile_collect(char* buf, size_t buflen)
{
    QLESS_REQUIRE(buf != nullptr && buflen > 0, QLESS_ERR_INVALID_ARG, "buf is required");
    struct Acc { const char* name; double ms; int count; };
    std::vector<Acc> acc;
    for (auto& r : t_prof) {
        float ms = 0.f;
        cudaEventSynchronize(r.b);
        if (cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) ms = 0.f;
        cudaEventDestroy(r.a); cudaEventDestroy(r.b);
        bool found = false;
        for (auto& a : acc) if (strcmp(a.name, r.name) == 0) { a.ms += ms; a.count++; found = true; break; }
        if (!found) acc.push_back({r.name, ms, 1});
    }
    t_prof.clear();
    size_t pos = 0;
    buf[0] = 0;
    for (auto& a : acc) {
        int w = snprintf(buf + pos, buflen - pos, "%s=%.6f*%d;", a.name, a.ms, a.count);
        if (w < 0 || (size_t)w >= buflen - pos) break;
        pos += (size_t)w;
    }
    return QLESS_OK;
}

size_t qless_project_quantize_workspace(int64_t n, int64_t P, int32_t d, int32_t bits)
{
    (void)bits;
    if (n <= 0 || P <= 0 || d <= 0) return 256;
    return pq_layout(n, P, d).total;
}

qless_status qless_project_quantize(const void* grads, qless_dtype dtype, int64_t n, int64_t ld_grads,
                                    const float* adam_m, const float* adam_v, const qless_adam_cfg* adam,
                                    int64_t P, int32_t d, uint64_t seed, int32_t bits, void* codes, float* scales,
                                    int32_t* code_sumsq, float* proj_out, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream)
{
    return qless_project_quantize_ex(grads, dtype, n, ld_grads, adam_m, adam_v, adam, P, d, seed, nullptr, bits, codes,
                                     scales, code_sumsq, proj_out, workspace, workspace_bytes, cuda_stream);
}

qless_status qless_project_quantize_ex(const void* grads, qless_dtype dtype, int64_t n, int64_t ld_grads,
                                       const float* adam_m, const float* adam_v, const qless_adam_cfg* adam,
                                       int64_t P, int32_t d, uint64_t seed, const qless_projection_cfg* projection,
                                       int32_t bits, void* codes, float* scales, int32_t* code_sumsq, float* proj_out,
                                       void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    qless_status s = check_grads(grads, dtype, n, ld_grads, adam_m, adam_v, P);
    if (s != QLESS_OK) return s;
    bool gaussian = false;
    s = matrix_kind(projection, &gaussian);
    if (s != QLESS_OK) return s;
    QLESS_REQUIRE(valid_bits(bits), QLESS_ERR_UNSUPPORTED, "bits must be 1, 2, 4 or 8 (bits=%d)", bits);
    QLESS_REQUIRE(d >= 128 && d <= 8192 && d % 128 == 0, QLESS_ERR_UNSUPPORTED, "d must be a multiple of 128 in [128, 8192] (d=%d)", d);
    AdamParams ap;
    s = make_adam(adam, &ap);
    if (s != QLESS_OK) return s;
    if (n == 0) return QLESS_OK;
    QLESS_REQUIRE(codes != nullptr && scales != nullptr, QLESS_ERR_INVALID_ARG, "codes and scales are required");
    QLESS_REQUIRE(aligned(codes, 16) && aligned(proj_out, 16), QLESS_ERR_INVALID_ARG, "codes and proj_out must be 16-byte aligned");
    const PqWorkspace w = pq_layout(n, P, d);
    QLESS_REQUIRE(workspace != nullptr && aligned(workspace, 256), QLESS_ERR_WORKSPACE, "workspace must be non-NULL and 256-byte aligned");
    QLESS_REQUIRE(workspace_bytes >= w.total, QLESS_ERR_WORKSPACE, "workspace too small: %zu bytes given, %zu needed", workspace_bytes, w.total);

    uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
    __nv_bfloat16* gamma = reinterpret_cast<__nv_bfloat16*>(ws + w.gamma_off);
    float* part = reinterpret_cast<float*>(ws + w.part_off);
    s = project_columns(grads, dtype, n, ld_grads, adam_m, adam_v, ap, w.plan, 0, P, seed, gaussian, gamma, part, st);
    if (s != QLESS_OK) return s;
    const float inv_sqrt_d = 1.0f / sqrtf((float)d);
    { ProfileScope ps("quantize", st);
      QLESS_CUDA_TRY(launch_quantize(part, w.plan.num_chunks, inv_sqrt_d, n, d, 1, bits, codes, scales, code_sumsq, proj_out, st)); }
    return QLESS_OK;
}

size_t qless_project_quantize_host_workspace(int64_t n, int64_t P, int32_t d, int32_t bits, qless_dtype dtype)
{
    if (n <= 0 || P <= 0 || d <= 0) return 256;
    const size_t esz = (dtype == QLESS_BF16) ? 2 : 4;
    return align_up((size_t)n * (size_t)P * esz, 256) + align_up((size_t)n * (size_t)d * bits / 8, 256) +
           2 * align_up((size_t)n * 4, 256) + qless_project_quantize_workspace(n, P, d, bits);
}

qless_status qless_project_quantize_host(const void* grads_host, qless_dtype dtype, int64_t n, int64_t ld_grads,
                                         const float* adam_m, const float* adam_v, const qless_adam_cfg* adam,
                                         int64_t P, int32_t d, uint64_t seed, int32_t bits, void* codes_host,
                                         float* scales_host, int32_t* code_sumsq_host, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream)
{
    return qless_project_quantize_host_ex(grads_host, dtype, n, ld_grads, adam_m, adam_v, adam, P, d, seed, nullptr, bits,
                                          codes_host, scales_host, code_sumsq_host, workspace, workspace_bytes, cuda_stream);
}

qless_status qless_project_quantize_host_ex(const void* grads_host, qless_dtype dtype, int64_t n, int64_t ld_grads,
                                            const float* adam_m, const float* adam_v, const qless_adam_cfg* adam,
                                            int64_t P, int32_t d, uint64_t seed, const qless_projection_cfg* projection,
                                            int32_t bits, void* codes_host, float* scales_host, int32_t* code_sumsq_host,
                                            void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    bool gaussian = false;
    { const qless_status ms = matrix_kind(projection, &gaussian); if (ms != QLESS_OK) return ms; }
    QLESS_REQUIRE(n >= 0 && P > 0 && d > 0, QLESS_ERR_INVALID_ARG, "n >= 0, P > 0, d > 0 required");
    QLESS_REQUIRE(dtype == QLESS_F32 || dtype == QLESS_BF16, QLESS_ERR_INVALID_ARG, "dtype must be QLESS_F32 or QLESS_BF16");
    QLESS_REQUIRE(valid_bits(bits), QLESS_ERR_UNSUPPORTED, "bits must be 1, 2, 4 or 8 (bits=%d)", bits);
    if (n == 0) return QLESS_OK;
    QLESS_REQUIRE(grads_host && codes_host && scales_host, QLESS_ERR_INVALID_ARG, "grads_host, codes_host and scales_host are required");
    QLESS_REQUIRE(ld_grads >= P, QLESS_ERR_INVALID_ARG, "ld_grads must be >= P");
    const size_t need = qless_project_quantize_host_workspace(n, P, d, bits, dtype);
    QLESS_REQUIRE(workspace != nullptr && aligned(workspace, 256), QLESS_ERR_WORKSPACE, "workspace must be non-NULL and 256-byte aligned");
    QLESS_REQUIRE(workspace_bytes >= need, QLESS_ERR_WORKSPACE, "workspace too small: %zu bytes given, %zu needed", workspace_bytes, need);
    const size_t esz = (dtype == QLESS_BF16) ? 2 : 4;
    uint8_t* p = reinterpret_cast<uint8_t*>(workspace);
    void* d_grads = p; p += align_up((size_t)n * (size_t)P * esz, 256);
    void* d_codes = p; p += align_up((size_t)n * (size_t)d * bits / 8, 256);
    float* d_scales = reinterpret_cast<float*>(p); p += align_up((size_t)n * 4, 256);
    int32_t* d_sumsq = reinterpret_cast<int32_t*>(p); p += align_up((size_t)n * 4, 256);
    const size_t inner = workspace_bytes - (size_t)(p - reinterpret_cast<uint8_t*>(workspace));
    // The batch crosses the host link in column slabs on a stream of the library's own; the prologue and the
    // projection of a slab run on the caller's stream while the next slab is copied. The staging buffer holds the
    // whole batch, so slabs never overwrite each other; the first copy waits for what the caller's stream had
    // queued before this call (an earlier call may still be reading the buffer).
    AdamParams ap;
    qless_status s = make_adam(adam, &ap);
    if (s != QLESS_OK) return s;
    QLESS_REQUIRE((adam_m == nullptr) == (adam_v == nullptr), QLESS_ERR_INVALID_ARG, "adam_m and adam_v must both be given or both be NULL");
    QLESS_REQUIRE(P % 128 == 0 && P < ((int64_t)1 << 39), QLESS_ERR_UNSUPPORTED, "P must be a multiple of 128 below 2^39 (P=%lld)", (long long)P);
    QLESS_REQUIRE(d >= 128 && d <= 8192 && d % 128 == 0, QLESS_ERR_UNSUPPORTED, "d must be a multiple of 128 in [128, 8192] (d=%d)", d);
    QLESS_REQUIRE(aligned(adam_m, 16) && aligned(adam_v, 16), QLESS_ERR_INVALID_ARG, "adam_m, adam_v must be 16-byte aligned");
    const PqWorkspace w = pq_layout(n, P, d);
    QLESS_REQUIRE(inner >= w.total, QLESS_ERR_WORKSPACE, "internal: workspace accounting");
    __nv_bfloat16* gamma = reinterpret_cast<__nv_bfloat16*>(p + w.gamma_off);
    float* part = reinterpret_cast<float*>(p + w.part_off);
    cudaStream_t cs = nullptr;
    s = copy_stream(&cs);
    if (s != QLESS_OK) return s;
    // about eight slabs, each a whole number of K chunks; the copies take longer than the projection, so only the
    // projection of the last slab is not hidden behind a copy: the last eighth is cut into slabs that halve in size
    int64_t chunks_per_slab = (w.plan.num_chunks + 7) / 8;
    if (chunks_per_slab < 1) chunks_per_slab = 1;
    cudaEvent_t ev_entry = nullptr, ev_slab = nullptr;
    QLESS_CUDA_TRY(cudaEventCreateWithFlags(&ev_entry, cudaEventDisableTiming));
    cudaError_t ce = cudaEventRecord(ev_entry, st);
    if (ce == cudaSuccess) ce = cudaStreamWaitEvent(cs, ev_entry, 0);
    cudaEventDestroy(ev_entry);             // released once the recorded work has completed
    if (ce != cudaSuccess) return cuda_fail(ce, "event set-up of the host path");
    for (int64_t j0 = 0, len = 0; j0 < P; j0 += len) {
        const int64_t chunks_left = (P - j0 + w.plan.chunk - 1) / w.plan.chunk;
        const int64_t take = chunks_left > chunks_per_slab ? chunks_per_slab : (chunks_left + 1) / 2;
        len = take * w.plan.chunk;
        if (len > P - j0) len = P - j0;
        ce = cudaMemcpy2DAsync(reinterpret_cast<uint8_t*>(d_grads) + (size_t)j0 * esz, (size_t)P * esz,
                               reinterpret_cast<const uint8_t*>(grads_host) + (size_t)j0 * esz, (size_t)ld_grads * esz,
                               (size_t)len * esz, (size_t)n, cudaMemcpyHostToDevice, cs);
        if (ce == cudaSuccess) ce = cudaEventCreateWithFlags(&ev_slab, cudaEventDisableTiming);
        if (ce != cudaSuccess) return cuda_fail(ce, "host-to-device copy of a column slab");
        ce = cudaEventRecord(ev_slab, cs);
        if (ce == cudaSuccess) ce = cudaStreamWaitEvent(st, ev_slab, 0);
        cudaEventDestroy(ev_slab);
        if (ce != cudaSuccess) return cuda_fail(ce, "ordering a column slab before its projection");
        s = project_columns(d_grads, dtype, n, P, adam_m, adam_v, ap, w.plan, j0, len, seed, gaussian, gamma, part, st);
        if (s != QLESS_OK) return s;
    }
    { ProfileScope ps("quantize", st);
      QLESS_CUDA_TRY(launch_quantize(part, w.plan.num_chunks, 1.0f / sqrtf((float)d), n, d, 1, bits, d_codes, d_scales,
                                     code_sumsq_host ? d_sumsq : nullptr, nullptr, st)); }
    QLESS_CUDA_TRY(cudaMemcpyAsync(codes_host, d_codes, (size_t)n * (size_t)d * bits / 8, cudaMemcpyDeviceToHost, st));
    QLESS_CUDA_TRY(cudaMemcpyAsync(scales_host, d_scales, (size_t)n * 4, cudaMemcpyDeviceToHost, st));
    if (code_sumsq_host)
        QLESS_CUDA_TRY(cudaMemcpyAsync(code_sumsq_host, d_sumsq, (size_t)n * 4, cudaMemcpyDeviceToHost, st));
    return QLESS_OK;
}

qless_status qless_quantize(const float* x, int64_t n, int32_t d, int32_t normalize, int32_t bits, void* codes,
                            float* scales, int32_t* code_sumsq, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(n >= 0, QLESS_ERR_INVALID_ARG, "n must be >= 0");
    QLESS_REQUIRE(valid_bits(bits), QLESS_ERR_UNSUPPORTED, "bits must be 1, 2, 4 or 8 (bits=%d)", bits);
    QLESS_REQUIRE(d >= 128 && d <= 8192 && d % 128 == 0, QLESS_ERR_UNSUPPORTED, "d must be a multiple of 128 in [128, 8192] (d=%d)", d);
    if (n == 0) return QLESS_OK;
    QLESS_REQUIRE(x != nullptr && codes != nullptr && scales != nullptr, QLESS_ERR_INVALID_ARG, "x, codes and scales are required");
    QLESS_REQUIRE(aligned(x, 16) && aligned(codes, 16), QLESS_ERR_INVALID_ARG, "x and codes must be 16-byte aligned");
    { ProfileScope ps("quantize", st);
      QLESS_CUDA_TRY(launch_quantize(x, 1, 1.0f, n, d, normalize ? 1 : 0, bits, codes, scales, code_sumsq, nullptr, st)); }
    return QLESS_OK;
}

qless_status qless_quantize_absmean(const float* x, int64_t n, int32_t d, int32_t normalize, int32_t bits, void* codes,
                                    float* scales, int32_t* code_sumsq, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(n >= 0, QLESS_ERR_INVALID_ARG, "n must be >= 0");
    QLESS_REQUIRE(valid_bits(bits), QLESS_ERR_UNSUPPORTED, "bits must be 1, 2, 4 or 8 (bits=%d)", bits);
    QLESS_REQUIRE(d >= 128 && d <= 8192 && d % 128 == 0, QLESS_ERR_UNSUPPORTED, "d must be a multiple of 128 in [128, 8192] (d=%d)", d);
    if (n == 0) return QLESS_OK;
    QLESS_REQUIRE(x != nullptr && codes != nullptr && scales != nullptr, QLESS_ERR_INVALID_ARG, "x, codes and scales are required");
    QLESS_REQUIRE(aligned(x, 16) && aligned(codes, 16), QLESS_ERR_INVALID_ARG, "x and codes must be 16-byte aligned");
    { ProfileScope ps("quantize_absmean", st);
      QLESS_CUDA_TRY(launch_quantize_absmean(x, n, d, normalize ? 1 : 0, bits, codes, scales, code_sumsq, st)); }
    return QLESS_OK;
}

qless_status qless_adam_gamma(const void* grads, qless_dtype dtype, int64_t n, int64_t ld_grads, const float* adam_m,
                              const float* adam_v, const qless_adam_cfg* adam, int64_t P, void* gamma_out,
                              void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    qless_status s = check_grads(grads, dtype, n, ld_grads, adam_m, adam_v, P);
    if (s != QLESS_OK) return s;
    AdamParams ap;
    s = make_adam(adam, &ap);
    if (s != QLESS_OK) return s;
    if (n == 0) return QLESS_OK;
    QLESS_REQUIRE(gamma_out != nullptr && aligned(gamma_out, 16), QLESS_ERR_INVALID_ARG, "gamma_out must be non-NULL and 16-byte aligned");
    QLESS_CUDA_TRY(launch_adam_gamma(grads, dtype, n, ld_grads, adam_m, adam_v, ap, P,
                                     reinterpret_cast<__nv_bfloat16*>(gamma_out), false, st));
    return QLESS_OK;
}

qless_status qless_philox_entries(uint64_t seed, int64_t r0, int64_t nr, int64_t j0, int64_t nj, int8_t* out,
                                  void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(r0 >= 0 && nr >= 0 && j0 >= 0 && nj >= 0, QLESS_ERR_INVALID_ARG, "negative range");
    QLESS_REQUIRE(r0 + nr <= ((int64_t)1 << 32) && j0 + nj <= ((int64_t)1 << 39), QLESS_ERR_UNSUPPORTED, "row < 2^32 and column < 2^39 required");
    if (nr == 0 || nj == 0) return QLESS_OK;
    QLESS_REQUIRE(out != nullptr, QLESS_ERR_INVALID_ARG, "out is NULL");
    QLESS_CUDA_TRY(launch_philox_entries(seed, r0, nr, j0, nj, out, st));
    return QLESS_OK;
}

// ---- scoring -----------------------------------------------------------------------------------

static qless_status check_score_shape(int64_t N, int32_t V, int32_t d, int32_t bits)
{
    QLESS_REQUIRE(N >= 0, QLESS_ERR_INVALID_ARG, "N must be >= 0");
    QLESS_REQUIRE(valid_bits(bits), QLESS_ERR_UNSUPPORTED, "bits must be 1, 2, 4 or 8 (bits=%d)", bits);
    QLESS_REQUIRE(d >= 128 && d <= 8192 && d % 128 == 0, QLESS_ERR_UNSUPPORTED, "d must be a multiple of 128 in [128, 8192] (d=%d)", d);
    QLESS_REQUIRE(V >= 1 && V <= 4096, QLESS_ERR_UNSUPPORTED, "V must be in [1, 4096] (V=%d)", V);
    return QLESS_OK;
}

struct ScoreWs { size_t tmult, vmult, eta, off, vunp, total; };
static ScoreWs score_layout(int64_t N, int32_t V, int32_t C, int32_t T, int32_t d, int32_t bits)
{
    ScoreWs w;
    w.tmult = 0;
    w.vmult = w.tmult + align_up((size_t)C * (size_t)N * 4, 256);
    w.eta = w.vmult + align_up((size_t)C * (size_t)V * 4, 256);
    w.off = w.eta + align_up((size_t)C * (size_t)T * 4, 256);
    w.vunp = w.off + align_up((size_t)(T + 1) * 4, 256);
    w.total = w.vunp + score_tc_workspace_bytes(V, C, d, bits);
    return w;
}

size_t qless_score_workspace(int64_t N, int32_t V, int32_t C, int32_t T, int32_t d, int32_t bits)
{
    if (N < 0 || V <= 0 || C <= 0 || T <= 0 || d <= 0) return 256;
    return score_layout(N, V, C, T, d, bits).total;
}

qless_status qless_score(const void* train_codes, int64_t train_ckpt_stride_bytes, const void* val_codes,
                         int64_t val_ckpt_stride_bytes, const float* train_scales, const float* val_scales,
                         const int32_t* train_sumsq, const int32_t* val_sumsq, const float* lr_weights,
                         const int32_t* task_offsets, int64_t N, int32_t V, int32_t C, int32_t T, int32_t d,
                         int32_t bits, qless_score_mode mode, float* scores, float* per_task, void* workspace,
                         size_t workspace_bytes, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    qless_status s = check_score_shape(N, V, d, bits);
    if (s != QLESS_OK) return s;
    QLESS_REQUIRE(C >= 1 && C <= 64, QLESS_ERR_UNSUPPORTED, "C must be in [1, 64] (C=%d)", C);
    QLESS_REQUIRE(T >= 1 && T <= 64, QLESS_ERR_UNSUPPORTED, "T must be in [1, 64] (T=%d)", T);
    QLESS_REQUIRE(mode == QLESS_SCORE_COSINE || mode == QLESS_SCORE_DEQUANT, QLESS_ERR_INVALID_ARG, "unknown score mode");
    QLESS_REQUIRE(lr_weights != nullptr && task_offsets != nullptr, QLESS_ERR_INVALID_ARG, "lr_weights and task_offsets (host) are required");
    QLESS_REQUIRE(task_offsets[0] == 0 && task_offsets[T] == V, QLESS_ERR_INVALID_ARG, "task_offsets must start at 0 and end at V");
    for (int j = 0; j < T; ++j)
        QLESS_REQUIRE(task_offsets[j + 1] > task_offsets[j], QLESS_ERR_INVALID_ARG, "task_offsets must be strictly increasing (task %d)", j);
    const int64_t row_bytes = (int64_t)d * bits / 8;
    QLESS_REQUIRE(train_ckpt_stride_bytes >= N * row_bytes && train_ckpt_stride_bytes % 16 == 0 &&
                  val_ckpt_stride_bytes >= V * row_bytes && val_ckpt_stride_bytes % 16 == 0,
                  QLESS_ERR_INVALID_ARG, "checkpoint strides must cover a checkpoint and be multiples of 16");
    if (N == 0) return QLESS_OK;
    QLESS_REQUIRE(train_codes && val_codes && train_scales && val_scales && scores, QLESS_ERR_INVALID_ARG, "codes, scales and scores are required");
    QLESS_REQUIRE(aligned(train_codes, 16) && aligned(val_codes, 16), QLESS_ERR_INVALID_ARG, "code arrays must be 16-byte aligned");
    const ScoreWs w = score_layout(N, V, C, T, d, bits);
    QLESS_REQUIRE(workspace != nullptr && aligned(workspace, 256), QLESS_ERR_WORKSPACE, "workspace must be non-NULL and 256-byte aligned");
    QLESS_REQUIRE(workspace_bytes >= w.total, QLESS_ERR_WORKSPACE, "workspace too small: %zu bytes given, %zu needed", workspace_bytes, w.total);

    uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
    float* tmult = reinterpret_cast<float*>(ws + w.tmult);
    float* vmult = reinterpret_cast<float*>(ws + w.vmult);
    float* d_eta = reinterpret_cast<float*>(ws + w.eta);
    int32_t* d_off = reinterpret_cast<int32_t*>(ws + w.off);

    std::vector<float> eoc((size_t)C * T);
    for (int i = 0; i < C; ++i)
        for (int j = 0; j < T; ++j)
            eoc[(size_t)i * T + j] = lr_weights[i] / (float)(task_offsets[j + 1] - task_offsets[j]);
    // pageable host sources: the runtime stages them before returning, so the vectors may die here
    QLESS_CUDA_TRY(cudaMemcpyAsync(d_eta, eoc.data(), eoc.size() * 4, cudaMemcpyHostToDevice, st));
    QLESS_CUDA_TRY(cudaMemcpyAsync(d_off, task_offsets, (size_t)(T + 1) * 4, cudaMemcpyHostToDevice, st));
    QLESS_CUDA_TRY(launch_multipliers(reinterpret_cast<const uint8_t*>(train_codes), train_ckpt_stride_bytes, train_scales,
                                      train_sumsq, N, C, d, bits, (int)mode, tmult, st));
    QLESS_CUDA_TRY(launch_multipliers(reinterpret_cast<const uint8_t*>(val_codes), val_ckpt_stride_bytes, val_scales,
                                      val_sumsq, V, C, d, bits, (int)mode, vmult, st));
    ScoreArgs a;
    a.train = reinterpret_cast<const uint8_t*>(train_codes); a.train_stride = train_ckpt_stride_bytes;
    a.val = reinterpret_cast<const uint8_t*>(val_codes); a.val_stride = val_ckpt_stride_bytes;
    a.train_mult = tmult; a.val_mult = vmult; a.eta_over_cnt = d_eta; a.task_off = d_off;
    a.N = N; a.V = V; a.C = C; a.T = T; a.d = d; a.bits = bits;
    a.scores = scores; a.per_task = per_task; a.dots = nullptr;
    if (g_score_path == 0 && score_tc_supported(T)) {
        unsigned int* flag = timeout_flag_ptr();
        QLESS_REQUIRE(flag != nullptr, QLESS_ERR_CUDA, "cannot resolve the device timeout flag");
        ProfileScope ps("score", st);
        s = launch_score_tc(a, ws + w.vunp, flag, st);
        if (s != QLESS_OK) return s;
    } else {
        ProfileScope ps("score", st);
        QLESS_CUDA_TRY(launch_score_simt(a, st));
    }
    return QLESS_OK;
}

size_t qless_score_16bit_workspace(int64_t N, int32_t V, int32_t C, int32_t T)
{
    if (N < 0 || V <= 0 || C <= 0 || T <= 0) return 256;
    return score_layout(N, V, C, T, 128, 8).total;
}

qless_status qless_inv_norms_16bit(const void* rows, int64_t ckpt_stride_bytes, int64_t nrows, int32_t C, int32_t d,
                                   float* inv_norms, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(nrows >= 0 && C >= 1, QLESS_ERR_INVALID_ARG, "nrows >= 0 and C >= 1 required");
    QLESS_REQUIRE(d >= 128 && d <= 8192 && d % 128 == 0, QLESS_ERR_UNSUPPORTED, "d must be a multiple of 128 in [128, 8192] (d=%d)", d);
    QLESS_REQUIRE(ckpt_stride_bytes >= nrows * (int64_t)d * 2 && ckpt_stride_bytes % 16 == 0, QLESS_ERR_INVALID_ARG,
                  "checkpoint stride must cover a checkpoint and be a multiple of 16");
    if (nrows == 0) return QLESS_OK;
    QLESS_REQUIRE(rows != nullptr && inv_norms != nullptr && aligned(rows, 16), QLESS_ERR_INVALID_ARG, "rows (16-byte aligned) and inv_norms are required");
    QLESS_CUDA_TRY(launch_inv_norms_bf16(reinterpret_cast<const uint8_t*>(rows), ckpt_stride_bytes, nrows, C, d, inv_norms, st));
    return QLESS_OK;
}

qless_status qless_score_16bit(const void* train_rows, int64_t train_ckpt_stride_bytes, const void* val_rows,
                               int64_t val_ckpt_stride_bytes, const float* train_inv_norms, const float* val_inv_norms,
                               const float* lr_weights, const int32_t* task_offsets,
                               int64_t N, int32_t V, int32_t C, int32_t T, int32_t d, float* scores, float* per_task,
                               void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    qless_status s = check_score_shape(N, V, d, 8);
    if (s != QLESS_OK) return s;
    QLESS_REQUIRE(C >= 1 && C <= 64, QLESS_ERR_UNSUPPORTED, "C must be in [1, 64] (C=%d)", C);
    QLESS_REQUIRE(T >= 1 && T <= 8, QLESS_ERR_UNSUPPORTED, "T must be in [1, 8] (T=%d)", T);
    QLESS_REQUIRE(lr_weights != nullptr && task_offsets != nullptr, QLESS_ERR_INVALID_ARG, "lr_weights and task_offsets (host) are required");
    QLESS_REQUIRE(task_offsets[0] == 0 && task_offsets[T] == V, QLESS_ERR_INVALID_ARG, "task_offsets must start at 0 and end at V");
    for (int j = 0; j < T; ++j)
        QLESS_REQUIRE(task_offsets[j + 1] > task_offsets[j], QLESS_ERR_INVALID_ARG, "task_offsets must be strictly increasing (task %d)", j);
    const int64_t row_bytes = (int64_t)d * 2;
    QLESS_REQUIRE(train_ckpt_stride_bytes >= N * row_bytes && train_ckpt_stride_bytes % 16 == 0 &&
                  val_ckpt_stride_bytes >= V * row_bytes && val_ckpt_stride_bytes % 16 == 0,
                  QLESS_ERR_INVALID_ARG, "checkpoint strides must cover a checkpoint and be multiples of 16");
    if (N == 0) return QLESS_OK;
    QLESS_REQUIRE(train_rows && val_rows && scores, QLESS_ERR_INVALID_ARG, "train_rows, val_rows and scores are required");
    QLESS_REQUIRE(aligned(train_rows, 16) && aligned(val_rows, 16), QLESS_ERR_INVALID_ARG, "row arrays must be 16-byte aligned");
    const ScoreWs w = score_layout(N, V, C, T, 128, 8);
    QLESS_REQUIRE(workspace != nullptr && aligned(workspace, 256), QLESS_ERR_WORKSPACE, "workspace must be non-NULL and 256-byte aligned");
    QLESS_REQUIRE(workspace_bytes >= w.total, QLESS_ERR_WORKSPACE, "workspace too small: %zu bytes given, %zu needed", workspace_bytes, w.total);
    uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
    float* tmult = reinterpret_cast<float*>(ws + w.tmult);
    float* vmult = reinterpret_cast<float*>(ws + w.vmult);
    float* d_eta = reinterpret_cast<float*>(ws + w.eta);
    int32_t* d_off = reinterpret_cast<int32_t*>(ws + w.off);
    std::vector<float> eoc((size_t)C * T);
    for (int i = 0; i < C; ++i)
        for (int j = 0; j < T; ++j)
            eoc[(size_t)i * T + j] = lr_weights[i] / (float)(task_offsets[j + 1] - task_offsets[j]);
    QLESS_CUDA_TRY(cudaMemcpyAsync(d_eta, eoc.data(), eoc.size() * 4, cudaMemcpyHostToDevice, st));
    QLESS_CUDA_TRY(cudaMemcpyAsync(d_off, task_offsets, (size_t)(T + 1) * 4, cudaMemcpyHostToDevice, st));
    // the norms are a pass over the whole store: a caller that keeps them beside the store passes them in
    if (train_inv_norms == nullptr)
        QLESS_CUDA_TRY(launch_inv_norms_bf16(reinterpret_cast<const uint8_t*>(train_rows), train_ckpt_stride_bytes, N, C, d, tmult, st));
    if (val_inv_norms == nullptr)
        QLESS_CUDA_TRY(launch_inv_norms_bf16(reinterpret_cast<const uint8_t*>(val_rows), val_ckpt_stride_bytes, V, C, d, vmult, st));
    ScoreArgs a;
    a.train = reinterpret_cast<const uint8_t*>(train_rows); a.train_stride = train_ckpt_stride_bytes;
    a.val = reinterpret_cast<const uint8_t*>(val_rows); a.val_stride = val_ckpt_stride_bytes;
    a.train_mult = train_inv_norms ? train_inv_norms : tmult; a.val_mult = val_inv_norms ? val_inv_norms : vmult;
    a.eta_over_cnt = d_eta; a.task_off = d_off;
    a.N = N; a.V = V; a.C = C; a.T = T; a.d = d; a.bits = 16;
    a.scores = scores; a.per_task = per_task; a.dots = nullptr;
    unsigned int* flag = timeout_flag_ptr();
    QLESS_REQUIRE(flag != nullptr, QLESS_ERR_CUDA, "cannot resolve the device timeout flag");
    ProfileScope ps("score16", st);
    return launch_score_tc(a, nullptr, flag, st);
}

size_t qless_score_dots_workspace(int64_t nt, int32_t V, int32_t d, int32_t bits)
{
    (void)nt;
    if (V <= 0 || d <= 0) return 256;
    return 256 + score_tc_workspace_bytes(V, 1, d, bits);
}

qless_status qless_score_dots(const void* train_codes, const void* val_codes, int64_t t0, int64_t nt, int32_t V,
                              int32_t d, int32_t bits, int32_t* dots, void* workspace, size_t workspace_bytes,
                              void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    qless_status s = check_score_shape(nt, V, d, bits);
    if (s != QLESS_OK) return s;
    QLESS_REQUIRE(t0 >= 0, QLESS_ERR_INVALID_ARG, "t0 must be >= 0");
    if (nt == 0) return QLESS_OK;
    QLESS_REQUIRE(train_codes && val_codes && dots, QLESS_ERR_INVALID_ARG, "train_codes, val_codes and dots are required");
    QLESS_REQUIRE(aligned(train_codes, 16) && aligned(val_codes, 16), QLESS_ERR_INVALID_ARG, "code arrays must be 16-byte aligned");
    const int64_t row_bytes = (int64_t)d * bits / 8;
    ScoreArgs a;
    a.train = reinterpret_cast<const uint8_t*>(train_codes) + t0 * row_bytes; a.train_stride = 0;
    a.val = reinterpret_cast<const uint8_t*>(val_codes); a.val_stride = 0;
    a.train_mult = nullptr; a.val_mult = nullptr; a.eta_over_cnt = nullptr; a.task_off = nullptr;
    a.N = nt; a.V = V; a.C = 1; a.T = 1; a.d = d; a.bits = bits;
    a.scores = nullptr; a.per_task = nullptr; a.dots = dots;
    if (g_score_path == 0) {
        const size_t need = qless_score_dots_workspace(nt, V, d, bits);
        QLESS_REQUIRE(workspace != nullptr && aligned(workspace, 256), QLESS_ERR_WORKSPACE, "workspace must be non-NULL and 256-byte aligned");
        QLESS_REQUIRE(workspace_bytes >= need, QLESS_ERR_WORKSPACE, "workspace too small: %zu bytes given, %zu needed", workspace_bytes, need);
        unsigned int* flag = timeout_flag_ptr();
        QLESS_REQUIRE(flag != nullptr, QLESS_ERR_CUDA, "cannot resolve the device timeout flag");
        s = launch_score_tc(a, reinterpret_cast<uint8_t*>(workspace), flag, st);
        if (s != QLESS_OK) return s;
    } else {
        QLESS_CUDA_TRY(launch_score_simt(a, st));
    }
    return QLESS_OK;
}

// ---- selection ---------------------------------------------------------------------------------

size_t qless_select_topk_workspace(int64_t N) { return select_workspace_bytes(N); }

qless_status qless_select_topk(const float* scores, int64_t N, double frac, int64_t* indices, int64_t* k_out,
                               void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    QLESS_REQUIRE(N >= 0 && N < ((int64_t)1 << 31), QLESS_ERR_INVALID_ARG, "N must be in [0, 2^31)");
    QLESS_REQUIRE(frac >= 0.0 && frac <= 1.0, QLESS_ERR_INVALID_ARG, "frac must be in [0, 1]");   // also rejects NaN
    QLESS_REQUIRE(k_out != nullptr, QLESS_ERR_INVALID_ARG, "k_out (host) is required");
    double kf = std::floor(frac * (double)N + 1e-6);
    if (kf < 0.0) kf = 0.0;
    if (kf > (double)N) kf = (double)N;
    const int64_t k = (int64_t)kf;
    if (k > 0) {
        QLESS_REQUIRE(scores != nullptr && indices != nullptr, QLESS_ERR_INVALID_ARG, "scores and indices are required");
        QLESS_REQUIRE(aligned(scores, 16), QLESS_ERR_INVALID_ARG, "scores must be 16-byte aligned");
        QLESS_REQUIRE(workspace != nullptr && aligned(workspace, 256), QLESS_ERR_WORKSPACE, "workspace must be non-NULL and 256-byte aligned");
        QLESS_REQUIRE(workspace_bytes >= select_workspace_bytes(N), QLESS_ERR_WORKSPACE, "workspace too small: %zu bytes given, %zu needed",
                      workspace_bytes, select_workspace_bytes(N));
    }
    *k_out = k;
    if (k == 0) return QLESS_OK;
    { ProfileScope ps("select", st);
      QLESS_CUDA_TRY(launch_select_topk(scores, N, k, indices, workspace, st)); }
    return QLESS_OK;
}

}  // extern "C"
