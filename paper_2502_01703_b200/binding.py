"""Thin Python binding of the C ABI in ``include/qless.h``.

Every function has the name of the C entry point it calls and does argument marshalling only:
torch supplies device memory and the current CUDA stream, the arithmetic runs in the library's
kernels. If ``libqless.so`` has not been built, or a call returns a non-OK status, an exception is
raised; there is no other code path.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqless.so")

QLESS_OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 1, 2, 3, 4, 5
F32, BF16 = 0, 1
COSINE, DEQUANT = 0, 1

EXPORTS = [
    "qless_last_error", "qless_check", "qless_project_quantize_workspace", "qless_project_quantize",
    "qless_quantize", "qless_quantize_absmean", "qless_adam_gamma", "qless_philox_entries", "qless_score_workspace", "qless_score",
    "qless_score_16bit_workspace", "qless_score_16bit", "qless_inv_norms_16bit", "qless_score_dots_workspace", "qless_score_dots", "qless_select_topk_workspace", "qless_select_topk",
    "qless_project_quantize_host_workspace", "qless_project_quantize_host", "qless_profile_enable",
    "qless_profile_collect", "qless_kernel_launches", "qless_select_topk_static",
    "qless_set_projection_path", "qless_set_score_path", "qless_set_select_path", "qless_microbench",
    "qless_project_quantize_ex", "qless_project_quantize_host_ex", "qless_gaussian_entries", "qless_selftest_timeout",
]
RADEMACHER, GAUSSIAN = 0, 1
SELECT_STATIC_MAX_N = 1 << 22


class AdamCfg(C.Structure):
    _fields_ = [("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("step", C.c_int64)]


class ProjectionCfg(C.Structure):
    _fields_ = [("matrix", C.c_int32), ("reserved", C.c_int32 * 3)]


class QlessError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"qless status {status}: {message}")
        self.status = status


_lib = None


def lib():
    """The loaded shared library (loads it on first use; raises if it is missing)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build the CUDA library first (python -m paper_2502_01703_b200.build)")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32, u64, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_size_t
        L.qless_last_error.restype = C.c_char_p
        L.qless_last_error.argtypes = []
        L.qless_check.restype = C.c_int
        L.qless_check.argtypes = [vp]
        L.qless_project_quantize_workspace.restype = sz
        L.qless_project_quantize_workspace.argtypes = [i64, i64, i32, i32]
        L.qless_project_quantize.restype = C.c_int
        L.qless_project_quantize.argtypes = [vp, C.c_int, i64, i64, vp, vp, C.POINTER(AdamCfg), i64, i32, u64, i32,
                                             vp, vp, vp, vp, vp, sz, vp]
        L.qless_project_quantize_host_workspace.restype = sz
        L.qless_project_quantize_host_workspace.argtypes = [i64, i64, i32, i32, C.c_int]
        L.qless_project_quantize_host.restype = C.c_int
        L.qless_project_quantize_host.argtypes = [vp, C.c_int, i64, i64, vp, vp, C.POINTER(AdamCfg), i64, i32, u64, i32,
                                                  vp, vp, vp, vp, sz, vp]
        L.qless_profile_enable.restype = C.c_int
        L.qless_profile_enable.argtypes = [i32]
        L.qless_kernel_launches.restype = C.c_uint64
        L.qless_kernel_launches.argtypes = []
        L.qless_profile_collect.restype = C.c_int
        L.qless_profile_collect.argtypes = [C.c_char_p, sz]
        L.qless_quantize.restype = C.c_int
        L.qless_quantize.argtypes = [vp, i64, i32, i32, i32, vp, vp, vp, vp]
        L.qless_quantize_absmean.restype = C.c_int
        L.qless_quantize_absmean.argtypes = [vp, i64, i32, i32, i32, vp, vp, vp, vp]
        L.qless_adam_gamma.restype = C.c_int
        L.qless_adam_gamma.argtypes = [vp, C.c_int, i64, i64, vp, vp, C.POINTER(AdamCfg), i64, vp, vp]
        L.qless_philox_entries.restype = C.c_int
        L.qless_philox_entries.argtypes = [u64, i64, i64, i64, i64, vp, vp]
        L.qless_score_workspace.restype = sz
        L.qless_score_workspace.argtypes = [i64, i32, i32, i32, i32, i32]
        L.qless_score.restype = C.c_int
        L.qless_score.argtypes = [vp, i64, vp, i64, vp, vp, vp, vp, C.POINTER(C.c_float), C.POINTER(i32),
                                  i64, i32, i32, i32, i32, i32, C.c_int, vp, vp, vp, sz, vp]
        L.qless_score_16bit_workspace.restype = sz
        L.qless_score_16bit_workspace.argtypes = [i64, i32, i32, i32]
        L.qless_score_16bit.restype = C.c_int
        L.qless_score_16bit.argtypes = [vp, i64, vp, i64, vp, vp, C.POINTER(C.c_float), C.POINTER(i32), i64, i32, i32, i32,
                                        i32, vp, vp, vp, sz, vp]
        L.qless_inv_norms_16bit.restype = C.c_int
        L.qless_inv_norms_16bit.argtypes = [vp, i64, i64, i32, i32, vp, vp]
        L.qless_score_dots_workspace.restype = sz
        L.qless_score_dots_workspace.argtypes = [i64, i32, i32, i32]
        L.qless_score_dots.restype = C.c_int
        L.qless_score_dots.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, vp, sz, vp]
        L.qless_select_topk_workspace.restype = sz
        L.qless_select_topk_workspace.argtypes = [i64]
        L.qless_select_topk.restype = C.c_int
        L.qless_select_topk.argtypes = [vp, i64, C.c_double, vp, C.POINTER(i64), vp, sz, vp]
        L.qless_microbench.restype = C.c_int
        L.qless_microbench.argtypes = [i32, i32, C.POINTER(C.c_float), C.POINTER(C.c_double), vp, sz, vp]
        L.qless_set_score_path.restype = C.c_int
        L.qless_set_score_path.argtypes = [i32]
        L.qless_set_select_path.restype = C.c_int
        L.qless_set_select_path.argtypes = [i32]
        L.qless_set_projection_path.restype = C.c_int
        L.qless_set_projection_path.argtypes = [i32]
        L.qless_project_quantize_ex.restype = C.c_int
        L.qless_project_quantize_ex.argtypes = [vp, C.c_int, i64, i64, vp, vp, C.POINTER(AdamCfg), i64, i32, u64,
                                                C.POINTER(ProjectionCfg), i32, vp, vp, vp, vp, vp, sz, vp]
        L.qless_project_quantize_host_ex.restype = C.c_int
        L.qless_project_quantize_host_ex.argtypes = [vp, C.c_int, i64, i64, vp, vp, C.POINTER(AdamCfg), i64, i32, u64,
                                                     C.POINTER(ProjectionCfg), i32, vp, vp, vp, vp, sz, vp]
        L.qless_selftest_timeout.restype = C.c_int
        L.qless_selftest_timeout.argtypes = [i32, vp]
        L.qless_gaussian_entries.restype = C.c_int
        L.qless_gaussian_entries.argtypes = [C.c_uint64, i64, i64, i64, i64, vp, vp]
        L.qless_select_topk_static.restype = C.c_int
        L.qless_select_topk_static.argtypes = [vp, i64, C.c_double, vp, C.POINTER(i64), vp]
        _lib = L
    return _lib


def _check(status):
    if status != QLESS_OK:
        raise QlessError(status, lib().qless_last_error().decode())


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _dtype_code(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("gradients must be float32 or bfloat16")


def _adam(adam):
    if adam is None:
        return None
    return C.byref(AdamCfg(adam.get("beta1", 0.9), adam.get("beta2", 0.999), adam.get("eps", 1e-8),
                           int(adam.get("step", 0))))


def _projection(matrix):
    return C.byref(ProjectionCfg(int(matrix), (C.c_int32 * 3)(0, 0, 0)))


def _workspace(nbytes, device, workspace):
    if workspace is not None:
        return workspace
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def qless_last_error():
    return lib().qless_last_error().decode()


def qless_check(stream=None):
    _check(lib().qless_check(_stream(stream)))


def qless_project_quantize_workspace(n, P, d, bits):
    return int(lib().qless_project_quantize_workspace(n, P, d, bits))


def qless_project_quantize(grads, d, seed, bits, adam_m=None, adam_v=None, adam=None, want_sumsq=True,
                           want_proj=False, out=None, workspace=None, stream=None, matrix=None):
    """grads [n, P] f32/bf16 (row stride allowed) -> dict(codes uint8 [n, d*bits/8], scales f32 [n],
    sumsq i32 [n] | None, proj f32 [n, d] | None). `out` may pass preallocated tensors by those names.
    matrix = None calls qless_project_quantize; RADEMACHER / GAUSSIAN call qless_project_quantize_ex with that
    matrix in its projection config."""
    n, P = grads.shape
    dev = grads.device
    out = out or {}
    codes = out.get("codes", None)
    if codes is None:
        codes = torch.empty((n, d * bits // 8), dtype=torch.uint8, device=dev)
    scales = out.get("scales", None)
    if scales is None:
        scales = torch.empty(n, dtype=torch.float32, device=dev)
    sumsq = out.get("sumsq", torch.empty(n, dtype=torch.int32, device=dev) if want_sumsq else None)
    proj = out.get("proj", torch.empty((n, d), dtype=torch.float32, device=dev) if want_proj else None)
    ws = _workspace(qless_project_quantize_workspace(n, P, d, bits), dev, workspace)
    if matrix is None:
        _check(lib().qless_project_quantize(_ptr(grads), _dtype_code(grads), n, grads.stride(0) if n > 0 else P,
                                            _ptr(adam_m), _ptr(adam_v), _adam(adam), P, d, seed, bits,
                                            _ptr(codes), _ptr(scales), _ptr(sumsq), _ptr(proj),
                                            _ptr(ws), ws.numel(), _stream(stream)))
    else:
        _check(lib().qless_project_quantize_ex(_ptr(grads), _dtype_code(grads), n, grads.stride(0) if n > 0 else P,
                                               _ptr(adam_m), _ptr(adam_v), _adam(adam), P, d, seed, _projection(matrix),
                                               bits, _ptr(codes), _ptr(scales), _ptr(sumsq), _ptr(proj),
                                               _ptr(ws), ws.numel(), _stream(stream)))
    return dict(codes=codes, scales=scales, sumsq=sumsq, proj=proj)


def qless_project_quantize_host_workspace(n, P, d, bits, dtype_code):
    return int(lib().qless_project_quantize_host_workspace(n, P, d, bits, dtype_code))


def qless_project_quantize_host(grads_host, d, seed, bits, adam_m=None, adam_v=None, adam=None, out=None,
                                workspace=None, device="cuda", stream=None, matrix=None):
    """grads_host: CPU tensor [n, P] (pinned for asynchronous copies); adam_m / adam_v: device tensors.
    Returns dict(codes, scales, sumsq) of CPU tensors (pinned), valid once the stream has drained."""
    n, P = grads_host.shape
    out = out or {}
    codes = out.get("codes")
    if codes is None:
        codes = torch.empty((n, d * bits // 8), dtype=torch.uint8).pin_memory()
    scales = out.get("scales")
    if scales is None:
        scales = torch.empty(n, dtype=torch.float32).pin_memory()
    sumsq = out.get("sumsq")
    if sumsq is None:
        sumsq = torch.empty(n, dtype=torch.int32).pin_memory()
    code = _dtype_code(grads_host)
    ws = _workspace(qless_project_quantize_host_workspace(n, P, d, bits, code), device, workspace)
    if matrix is None:
        _check(lib().qless_project_quantize_host(_ptr(grads_host), code, n, grads_host.stride(0) if n > 0 else P,
                                                 _ptr(adam_m), _ptr(adam_v), _adam(adam), P, d, seed, bits,
                                                 _ptr(codes), _ptr(scales), _ptr(sumsq), _ptr(ws), ws.numel(),
                                                 _stream(stream)))
    else:
        _check(lib().qless_project_quantize_host_ex(_ptr(grads_host), code, n, grads_host.stride(0) if n > 0 else P,
                                                    _ptr(adam_m), _ptr(adam_v), _adam(adam), P, d, seed,
                                                    _projection(matrix), bits, _ptr(codes), _ptr(scales), _ptr(sumsq),
                                                    _ptr(ws), ws.numel(), _stream(stream)))
    return dict(codes=codes, scales=scales, sumsq=sumsq)


def qless_profile_enable(on=True):
    _check(lib().qless_profile_enable(1 if on else 0))


def qless_kernel_launches():
    return int(lib().qless_kernel_launches())


def qless_profile_collect():
    """{kernel name: (total milliseconds, launches)} since the last collect."""
    buf = C.create_string_buffer(4096)
    _check(lib().qless_profile_collect(buf, 4096))
    out = {}
    for item in buf.value.decode().split(";"):
        if item:
            name, rest = item.split("=")
            ms, cnt = rest.split("*")
            out[name] = (float(ms), int(cnt))
    return out


def qless_quantize(x, bits, normalize=True, want_sumsq=True, stream=None):
    n, d = x.shape
    dev = x.device
    codes = torch.empty((n, d * bits // 8), dtype=torch.uint8, device=dev)
    scales = torch.empty(n, dtype=torch.float32, device=dev)
    sumsq = torch.empty(n, dtype=torch.int32, device=dev) if want_sumsq else None
    _check(lib().qless_quantize(_ptr(x), n, d, 1 if normalize else 0, bits, _ptr(codes), _ptr(scales),
                                _ptr(sumsq), _stream(stream)))
    return codes, scales, sumsq


def qless_quantize_absmean(x, bits, normalize=True, want_sumsq=True, stream=None):
    """As qless_quantize, with the scale taken from the mean absolute value of the row."""
    n, d = x.shape
    dev = x.device
    codes = torch.empty((n, d * bits // 8), dtype=torch.uint8, device=dev)
    scales = torch.empty(n, dtype=torch.float32, device=dev)
    sumsq = torch.empty(n, dtype=torch.int32, device=dev) if want_sumsq else None
    _check(lib().qless_quantize_absmean(_ptr(x), n, d, 1 if normalize else 0, bits, _ptr(codes), _ptr(scales),
                                        _ptr(sumsq), _stream(stream)))
    return codes, scales, sumsq


def qless_adam_gamma(grads, adam_m=None, adam_v=None, adam=None, stream=None):
    n, P = grads.shape
    out = torch.empty((n, P), dtype=torch.bfloat16, device=grads.device)
    _check(lib().qless_adam_gamma(_ptr(grads), _dtype_code(grads), n, grads.stride(0) if n > 0 else P,
                                  _ptr(adam_m), _ptr(adam_v), _adam(adam), P, _ptr(out), _stream(stream)))
    return out


def qless_philox_entries(seed, r0, nr, j0, nj, device="cuda", stream=None):
    out = torch.empty((nr, nj), dtype=torch.int8, device=device)
    _check(lib().qless_philox_entries(seed, r0, nr, j0, nj, _ptr(out), _stream(stream)))
    return out


def qless_gaussian_entries(seed, r0, nr, j0, nj, device="cuda", stream=None):
    out = torch.empty((nr, nj), dtype=torch.float32, device=device)
    _check(lib().qless_gaussian_entries(seed, r0, nr, j0, nj, _ptr(out), _stream(stream)))
    return out


def qless_score_workspace(N, V, Cn, T, d, bits):
    return int(lib().qless_score_workspace(N, V, Cn, T, d, bits))


def qless_score(train_codes, val_codes, train_scales, val_scales, lr_weights, task_offsets, d, bits,
                train_sumsq=None, val_sumsq=None, mode=COSINE, want_per_task=False, scores=None,
                workspace=None, stream=None):
    """train_codes uint8 [C, N, d*bits/8], val_codes uint8 [C, V, d*bits/8] (checkpoint stride taken from
    the tensors), scales f32 [C, N] / [C, V]; lr_weights / task_offsets: host sequences."""
    Cn, N, rb = train_codes.shape
    V = val_codes.shape[1]
    dev = train_codes.device
    T = len(task_offsets) - 1
    eta = (C.c_float * Cn)(*[float(x) for x in lr_weights])
    off = (C.c_int32 * (T + 1))(*[int(x) for x in task_offsets])
    if scores is None:
        scores = torch.empty(N, dtype=torch.float32, device=dev)
    per_task = torch.empty((N, T), dtype=torch.float32, device=dev) if want_per_task else None
    ws = _workspace(qless_score_workspace(N, V, Cn, T, d, bits), dev, workspace)
    _check(lib().qless_score(_ptr(train_codes), train_codes.stride(0) if Cn > 0 else 0,
                             _ptr(val_codes), val_codes.stride(0),
                             _ptr(train_scales), _ptr(val_scales), _ptr(train_sumsq), _ptr(val_sumsq),
                             eta, off, N, V, Cn, T, d, bits, mode, _ptr(scores), _ptr(per_task),
                             _ptr(ws), ws.numel(), _stream(stream)))
    return (scores, per_task) if want_per_task else scores


def qless_score_16bit_workspace(N, V, Cn, T):
    return int(lib().qless_score_16bit_workspace(N, V, Cn, T))


def qless_inv_norms_16bit(rows, stream=None):
    """rows bf16 [C, n, d] -> 1 / ||row|| as f32 [C, n] (0 for a zero row)."""
    Cn, n, d = rows.shape
    out = torch.empty((Cn, n), dtype=torch.float32, device=rows.device)
    _check(lib().qless_inv_norms_16bit(_ptr(rows), rows.stride(0) * 2, n, Cn, d, _ptr(out), _stream(stream)))
    return out


def qless_score_16bit(train_rows, val_rows, lr_weights, task_offsets, want_per_task=False, scores=None,
                      workspace=None, stream=None, train_inv_norms=None, val_inv_norms=None):
    """The 16-bit baseline: train_rows bf16 [C, N, d], val_rows bf16 [C, V, d] (checkpoint stride taken from the
    tensors); lr_weights / task_offsets: host sequences."""
    assert train_rows.dtype == torch.bfloat16 and val_rows.dtype == torch.bfloat16
    Cn, N, d = train_rows.shape
    V = val_rows.shape[1]
    dev = train_rows.device
    T = len(task_offsets) - 1
    eta = (C.c_float * Cn)(*[float(x) for x in lr_weights])
    off = (C.c_int32 * (T + 1))(*[int(x) for x in task_offsets])
    if scores is None:
        scores = torch.empty(N, dtype=torch.float32, device=dev)
    per_task = torch.empty((N, T), dtype=torch.float32, device=dev) if want_per_task else None
    ws = _workspace(qless_score_16bit_workspace(N, V, Cn, T), dev, workspace)
    _check(lib().qless_score_16bit(_ptr(train_rows), train_rows.stride(0) * 2 if Cn > 0 else 0, _ptr(val_rows),
                                   val_rows.stride(0) * 2, _ptr(train_inv_norms), _ptr(val_inv_norms), eta, off, N, V, Cn, T,
                                   d, _ptr(scores), _ptr(per_task),
                                   _ptr(ws), ws.numel(), _stream(stream)))
    return (scores, per_task) if want_per_task else scores


def qless_score_dots_workspace(nt, V, d, bits):
    return int(lib().qless_score_dots_workspace(nt, V, d, bits))


def qless_score_dots(train_codes, val_codes, d, bits, t0=0, nt=None, workspace=None, stream=None):
    """One checkpoint: train_codes uint8 [N, rb], val_codes uint8 [V, rb] -> int32 [nt, V]."""
    if nt is None:
        nt = train_codes.shape[0] - t0
    V = val_codes.shape[0]
    dev = train_codes.device
    dots = torch.empty((nt, V), dtype=torch.int32, device=dev)
    ws = _workspace(qless_score_dots_workspace(nt, V, d, bits), dev, workspace)
    _check(lib().qless_score_dots(_ptr(train_codes), _ptr(val_codes), t0, nt, V, d, bits, _ptr(dots),
                                  _ptr(ws), ws.numel(), _stream(stream)))
    return dots


def qless_select_topk_workspace(N):
    return int(lib().qless_select_topk_workspace(N))


def qless_select_topk(scores, frac, indices=None, workspace=None, stream=None):
    """scores f32 [N] -> int64 [k] ascending indices of the top floor(frac*N) scores."""
    N = scores.numel()
    dev = scores.device
    if indices is None:
        indices = torch.empty(max(N, 1), dtype=torch.int64, device=dev)
    ws = _workspace(qless_select_topk_workspace(N), dev, workspace)
    k = C.c_int64(0)
    _check(lib().qless_select_topk(_ptr(scores), N, float(frac), _ptr(indices), C.byref(k), _ptr(ws),
                                   ws.numel(), _stream(stream)))
    return indices[:k.value]


def qless_select_topk_static(scores, frac, indices, stream=None):
    """Allocation-free variant of qless_select_topk for N <= SELECT_STATIC_MAX_N: the scratch is a fixed
    array inside the library, so the caller passes only the input and a preallocated int64 `indices`
    tensor with room for k entries. Returns a view of the first k entries; nothing is allocated here
    either. Calls that overlap on the GPU share that array and must be serialised by the caller."""
    k = C.c_int64(0)
    _check(lib().qless_select_topk_static(_ptr(scores), scores.numel(), float(frac), _ptr(indices), C.byref(k),
                                          _stream(stream)))
    return indices[:k.value]


def qless_set_projection_path(path):
    """0 = tensor-core projection kernel (default), 1 = CUDA-core cross-check kernel."""
    _check(lib().qless_set_projection_path(int(path)))


def qless_selftest_timeout(polls=1024, stream=None):
    """Enqueues the bounded-wait self-test kernel; the next qless_check() on the stream raises ERR_TIMEOUT."""
    _check(lib().qless_selftest_timeout(int(polls), _stream(stream)))


def qless_set_select_path(path):
    """0 = by size (default), 1 = multi-pass select at every N, 2 = sampled bracket forced too high."""
    _check(lib().qless_set_select_path(int(path)))


def qless_set_score_path(path):
    """0 = tensor-core scoring kernel for 8/4/2-bit codes (default), 1 = CUDA-core kernel."""
    _check(lib().qless_set_score_path(int(path)))


MICROBENCH = {"bf16_ss": 0, "bf16_ts": 1, "i8_ss": 2, "bf16_ss_pair": 3, "bf16_ts_pair": 4, "i8_ss_pair": 5, "popc": 6, "i8_ts_pair": 7,
              "i8_ss_pair_n448": 8, "tma_l2_stream": 9, "i8_n448_with_tma": 10, "i8_n448_commit_per_block": 11, "i8_n448_streamed_operands": 12,
              "fp4_ss_pair_n448": 13, "fp4_ts_pair": 14}


def qless_microbench(what, iters, device="cuda", stream=None, scratch=None):
    """(milliseconds, operations) of one peak-rate micro-benchmark; `what` is a key of MICROBENCH. `scratch`: a
    uint8 device tensor of at least 4 MiB whose contents the streaming benchmarks read (default: uninitialised)."""
    ms, ops = C.c_float(0), C.c_double(0)
    if scratch is None:
        scratch = torch.empty(4 << 20, dtype=torch.uint8, device=device)
    _check(lib().qless_microbench(MICROBENCH[what], int(iters), C.byref(ms), C.byref(ops), _ptr(scratch), scratch.numel(),
                                  _stream(stream)))
    return ms.value, ops.value
