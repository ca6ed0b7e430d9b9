"""numpy front end of the QLESS CPU oracle (oracle/qless_oracle.c).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does, and this
package never imports the CUDA library. Every function here only marshals numpy
arrays into the C routine of the same name; the arithmetic is in the C file,
each routine citing the equation of the paper it restates. Two functions are plain numpy instead, written out
below: score_16bit (Eq. 3) and quantize_absmean_rows. The latter is PARITY UNPINNED as far as the formula goes:
the paper names absmean quantisation (Sec. 6, Table 3) without giving it, so the function states one reading and
is pinned only to what the paper and the arithmetic fix (see its docstring).
"""
import ctypes as C
import os

import numpy as np

from .build import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _declare(_lib)
    return _lib


_u32p = C.POINTER(C.c_uint32)
_i8p = C.POINTER(C.c_int8)
_u8p = C.POINTER(C.c_uint8)
_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)
_f32p = C.POINTER(C.c_float)


def _declare(L):
    L.qlo_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
    L.qlo_philox4x32_10.restype = None
    L.qlo_rademacher_sign.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
    L.qlo_rademacher_sign.restype = C.c_int
    L.qlo_rademacher_row.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64, _i8p]
    L.qlo_rademacher_row.restype = None
    L.qlo_round_to_bf16.argtypes = [C.c_float]
    L.qlo_round_to_bf16.restype = C.c_float
    L.qlo_adam_gamma.argtypes = [_f32p, _f32p, _f32p, C.c_int64, C.c_float, C.c_float, C.c_float,
                                 C.c_int64, _f32p]
    L.qlo_adam_gamma.restype = None
    L.qlo_project.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_int32, C.c_uint64, _f32p]
    L.qlo_project.restype = None
    L.qlo_project_rows.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_int32, C.c_uint64, _i32p,
                                   C.c_int32, _f32p]
    L.qlo_project_rows.restype = None
    L.qlo_gaussian_entry_exact.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
    L.qlo_gaussian_entry_exact.restype = C.c_double
    L.qlo_gaussian_row.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64, _f32p]
    L.qlo_gaussian_row.restype = None
    L.qlo_project_gaussian.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_int32, C.c_uint64, _f32p]
    L.qlo_project_gaussian.restype = None
    L.qlo_normalize.argtypes = [_f32p, C.c_int32, _f32p]
    L.qlo_normalize.restype = C.c_float
    L.qlo_quantize.argtypes = [_f32p, C.c_int32, C.c_int32, _i8p, _i32p]
    L.qlo_quantize.restype = C.c_float
    L.qlo_pack.argtypes = [_i8p, C.c_int32, C.c_int32, _u8p]
    L.qlo_pack.restype = None
    L.qlo_unpack.argtypes = [_u8p, C.c_int32, C.c_int32, _i8p]
    L.qlo_unpack.restype = None
    L.qlo_quantize_rows.argtypes = [_f32p, C.c_int64, C.c_int32, C.c_int32, C.c_int, _u8p, _f32p, _i32p]
    L.qlo_quantize_rows.restype = None
    L.qlo_dot.argtypes = [_i8p, _i8p, C.c_int32]
    L.qlo_dot.restype = C.c_int64
    L.qlo_dots.argtypes = [_u8p, _u8p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_int32, _i32p]
    L.qlo_dots.restype = None
    L.qlo_score.argtypes = [_u8p, C.c_int64, _u8p, C.c_int64, _f32p, _f32p, _f32p, _i32p,
                            C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                            C.c_int64, C.c_int64, _f32p, _f32p]
    L.qlo_score.restype = None
    L.qlo_topk_count.argtypes = [C.c_int64, C.c_double]
    L.qlo_topk_count.restype = C.c_int64
    L.qlo_select_topk.argtypes = [_f32p, C.c_int64, C.c_double, _i64p]
    L.qlo_select_topk.restype = C.c_int64
    L.qlo_project_quantize.argtypes = [_f32p, C.c_int64, C.c_int64, _f32p, _f32p, C.c_float, C.c_float,
                                       C.c_float, C.c_int64, C.c_int32, C.c_uint64, C.c_int32,
                                       _u8p, _f32p, _i32p, _f32p]
    L.qlo_project_quantize.restype = None


def _p(a, t):
    return a.ctypes.data_as(t) if a is not None else None


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


ADAM_DEFAULT = dict(beta1=0.9, beta2=0.999, eps=1e-8, step=0)


def philox4x32_10(ctr, key):
    ctr = _c(ctr, np.uint32); key = _c(key, np.uint32)
    out = np.empty(4, np.uint32)
    lib().qlo_philox4x32_10(_p(ctr, _u32p), _p(key, _u32p), _p(out, _u32p))
    return out


def rademacher_sign(seed, r, j):
    return int(lib().qlo_rademacher_sign(int(seed), int(r), int(j)))


def rademacher_rows(seed, r0, nr, j0, nj):
    """int8 [nr, nj]: signs s_{r,j} for r in [r0, r0+nr), j in [j0, j0+nj)."""
    out = np.empty((nr, nj), np.int8)
    for a in range(nr):
        lib().qlo_rademacher_row(int(seed), int(r0 + a), int(j0), int(nj), _p(out[a], _i8p))
    return out


def round_to_bf16(x):
    x = _c(x, np.float32)
    out = np.empty_like(x)
    f = lib().qlo_round_to_bf16
    flat_in, flat_out = x.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = f(float(flat_in[i]))
    return out


def adam_gamma(g, m=None, v=None, beta1=0.9, beta2=0.999, eps=1e-8, step=0):
    """fp32 [n, P] (or [P]) of bf16-representable values: Gamma for each row of g."""
    g = _c(g, np.float32)
    g2 = g.reshape(-1, g.shape[-1])
    m = _c(m, np.float32) if m is not None else None
    v = _c(v, np.float32) if v is not None else None
    out = np.empty_like(g2)
    for i in range(g2.shape[0]):
        lib().qlo_adam_gamma(_p(g2[i], _f32p), _p(m, _f32p), _p(v, _f32p), g2.shape[1],
                             beta1, beta2, eps, int(step), _p(out[i], _f32p))
    return out.reshape(g.shape)


def project(gamma, d, seed):
    gamma = _c(gamma, np.float32)
    n, P = gamma.shape
    y = np.empty((n, d), np.float32)
    lib().qlo_project(_p(gamma, _f32p), n, P, d, int(seed), _p(y, _f32p))
    return y


def gaussian_entry_exact(seed, r, j):
    """Entry z_{r,j} of the Gaussian matrix before its rounding to bf16 (float64)."""
    return float(lib().qlo_gaussian_entry_exact(int(seed), int(r), int(j)))


def gaussian_rows(seed, r0, nr, j0, nj):
    """fp32 [nr, nj]: the bf16-rounded entries z_{r,j} for r in [r0, r0+nr), j in [j0, j0+nj)."""
    out = np.empty((nr, nj), np.float32)
    for a in range(nr):
        lib().qlo_gaussian_row(int(seed), int(r0 + a), int(j0), int(nj), _p(out[a], _f32p))
    return out


def project_gaussian(gamma, d, seed):
    """Eq. 1 with the Gaussian matrix: fp32 [n, d]."""
    gamma = _c(gamma, np.float32)
    n, P = gamma.shape
    y = np.empty((n, d), np.float32)
    lib().qlo_project_gaussian(_p(gamma, _f32p), n, P, d, int(seed), _p(y, _f32p))
    return y


def project_rows(gamma, d, seed, rows):
    """Projection restricted to output coordinates `rows`: fp32 [n, len(rows)]."""
    gamma = _c(gamma, np.float32)
    rows = _c(rows, np.int32)
    n, P = gamma.shape
    y = np.empty((n, rows.size), np.float32)
    lib().qlo_project_rows(_p(gamma, _f32p), n, P, d, int(seed), _p(rows, _i32p), rows.size, _p(y, _f32p))
    return y


def normalize(y):
    """(yhat [d] fp32, norm fp32) for one vector."""
    y = _c(y, np.float32)
    out = np.empty_like(y)
    nrm = lib().qlo_normalize(_p(y, _f32p), y.size, _p(out, _f32p))
    return out, np.float32(nrm)


def quantize(x, bits):
    """(q int8 [d] unpacked, S fp32, sumsq int) for one vector."""
    x = _c(x, np.float32)
    q = np.empty(x.size, np.int8)
    ss = C.c_int32(0)
    S = lib().qlo_quantize(_p(x, _f32p), x.size, bits, _p(q, _i8p), C.byref(ss))
    return q, np.float32(S), int(ss.value)


def pack(q, bits):
    q = _c(q, np.int8)
    out = np.empty(q.size * bits // 8, np.uint8)
    lib().qlo_pack(_p(q, _i8p), q.size, bits, _p(out, _u8p))
    return out


def unpack(codes, d, bits):
    codes = _c(codes, np.uint8)
    q = np.empty(d, np.int8)
    lib().qlo_unpack(_p(codes, _u8p), d, bits, _p(q, _i8p))
    return q


def quantize_rows(x, bits, normalize=True):
    """(codes uint8 [n, d*bits/8], scales fp32 [n], sumsq int32 [n])."""
    x = _c(x, np.float32)
    n, d = x.shape
    codes = np.empty((n, d * bits // 8), np.uint8)
    scales = np.empty(n, np.float32)
    sumsq = np.empty(n, np.int32)
    lib().qlo_quantize_rows(_p(x, _f32p), n, d, bits, 1 if normalize else 0,
                            _p(codes, _u8p), _p(scales, _f32p), _p(sumsq, _i32p))
    return codes, scales, sumsq


ABSMEAN_STEP = {2: 1.0, 4: 0.5, 8: 1.0 / 32.0}      # quantisation step in units of the mean absolute value


def quantize_absmean_rows(x, bits, normalize=True):
    """Absmean variant of Eq. 4-5 (Sec. 6, Table 3; the paper gives no formula: PARITY UNPINNED, this is the
    reading): with yhat the (optionally L2-normalised, Eq. 2) row in fp32,
        gamma = fp32( sum_m |yhat_m| (in fp64) / d ),   Delta = gamma * c_b,  c_2 = 1, c_4 = 1/2, c_8 = 1/32,
        q_m   = clamp( round_half_even( fp32(yhat_m * fp32(1 / Delta)) ), -alpha, alpha ),  alpha = 2^(b-1) - 1,
    and the stored scale is S = fp32(alpha * Delta), so that q_m * S / alpha dequantises as for absmax codes.
    b = 2 is the ternary round-and-clip of x / mean|x|; the constants for b = 4, 8 put the clip point at
    3.5 and about 4 mean absolute values. b = 1 is the sign code of Eq. 5 (no scale enters). A zero row gives
    zero codes and S = 0. Returns (codes uint8 [n, d*bits/8], scales fp32 [n], sumsq int32 [n])."""
    x = _c(x, np.float32)
    n, d = x.shape
    if bits == 1:
        return quantize_rows(x, 1, normalize)
    alpha = 2 ** (bits - 1) - 1
    codes = np.empty((n, d * bits // 8), np.uint8)
    scales = np.empty(n, np.float32)
    sumsq = np.empty(n, np.int32)
    for r in range(n):
        yh = normalize_row(x[r]) if normalize else x[r]
        gamma = np.float32(np.abs(yh.astype(np.float64)).sum() / d)
        if not gamma > 0:
            codes[r] = 0; scales[r] = 0; sumsq[r] = 0
            continue
        delta = np.float32(gamma * np.float32(ABSMEAN_STEP[bits]))
        rcp = np.float32(1.0) / delta
        t = (yh * rcp).astype(np.float32)
        q = np.clip(np.rint(t), -alpha, alpha).astype(np.int8)
        codes[r] = pack(q, bits)
        scales[r] = np.float32(alpha) * delta
        sumsq[r] = int((q.astype(np.int64) ** 2).sum())
    return codes, scales, sumsq


def normalize_row(y):
    return normalize(y)[0]


def dot(a, b):
    a = _c(a, np.int8); b = _c(b, np.int8)
    return int(lib().qlo_dot(_p(a, _i8p), _p(b, _i8p), a.size))


def dots(train_codes, val_codes, d, bits, t0=0, nt=None):
    """int32 [nt, V]: integer dots of one checkpoint's train rows [t0, t0+nt) with all val rows."""
    train_codes = _c(train_codes, np.uint8); val_codes = _c(val_codes, np.uint8)
    if nt is None:
        nt = train_codes.shape[0] - t0
    V = val_codes.shape[0]
    out = np.empty((nt, V), np.int32)
    lib().qlo_dots(_p(train_codes, _u8p), _p(val_codes, _u8p), t0, nt, V, d, bits, _p(out, _i32p))
    return out


def score(train_codes, val_codes, train_scales, val_scales, eta, task_offsets, d, bits,
          mode=0, t0=0, nt=None, want_per_task=False):
    """train_codes uint8 [C, N, rb], val_codes uint8 [C, V, rb], scales fp32 [C, N] / [C, V]."""
    train_codes = _c(train_codes, np.uint8); val_codes = _c(val_codes, np.uint8)
    train_scales = _c(train_scales, np.float32); val_scales = _c(val_scales, np.float32)
    eta = _c(eta, np.float32); task_offsets = _c(task_offsets, np.int32)
    Cn, N, rb = train_codes.shape
    V = val_codes.shape[1]
    T = task_offsets.size - 1
    if nt is None:
        nt = N - t0
    scores = np.empty(nt, np.float32)
    per_task = np.empty((nt, T), np.float32) if want_per_task else None
    lib().qlo_score(_p(train_codes, _u8p), N * rb, _p(val_codes, _u8p), V * rb,
                    _p(train_scales, _f32p), _p(val_scales, _f32p), _p(eta, _f32p),
                    _p(task_offsets, _i32p), N, V, Cn, T, d, bits, mode, t0, nt,
                    _p(scores, _f32p), _p(per_task, _f32p))
    return (scores, per_task) if want_per_task else scores


def score_16bit(train, val, eta, task_offsets, want_per_task=False):
    """The 16-bit LESS baseline (Eq. 3 with the aggregation of Sec. 4.1), written out: train [C, N, d] and
    val [C, V, d] hold the stored vectors (values that a 16-bit store can hold, passed as floats);
    score[t] = max_j sum_i eta_i * mean_{v in task j} <x_t,i, x_v,i> / (||x_t,i|| ||x_v,i||), in fp64; a zero
    vector has cosine 0 with everything."""
    train = np.asarray(train, np.float64); val = np.asarray(val, np.float64)
    eta = np.asarray(eta, np.float64); off = np.asarray(task_offsets, np.int64)
    Cn, N, d = train.shape
    T = off.size - 1
    per_task = np.zeros((N, T), np.float64)
    for i in range(Cn):
        tn = np.sqrt((train[i] * train[i]).sum(axis=1)); vn = np.sqrt((val[i] * val[i]).sum(axis=1))
        inner = train[i] @ val[i].T
        denom = tn[:, None] * vn[None, :]
        cos = np.divide(inner, denom, out=np.zeros_like(inner), where=denom > 0)
        for j in range(T):
            per_task[:, j] += eta[i] * cos[:, off[j]:off[j + 1]].mean(axis=1)
    scores = per_task.max(axis=1)
    return (scores, per_task) if want_per_task else scores


def topk_count(N, frac):
    return int(lib().qlo_topk_count(int(N), float(frac)))


def select_topk(scores, frac):
    scores = _c(scores, np.float32)
    idx = np.empty(max(scores.size, 1), np.int64)
    k = lib().qlo_select_topk(_p(scores, _f32p), scores.size, float(frac), _p(idx, _i64p))
    return idx[:k].copy()


def project_quantize(g, d, seed, bits, m=None, v=None, beta1=0.9, beta2=0.999, eps=1e-8, step=0,
                     want_proj=False):
    """(codes, scales, sumsq[, proj]) for gradient rows g fp32 [n, P]."""
    g = _c(g, np.float32)
    n, P = g.shape
    m = _c(m, np.float32) if m is not None else None
    v = _c(v, np.float32) if v is not None else None
    codes = np.empty((n, d * bits // 8), np.uint8)
    scales = np.empty(n, np.float32)
    sumsq = np.empty(n, np.int32)
    proj = np.empty((n, d), np.float32) if want_proj else None
    lib().qlo_project_quantize(_p(g, _f32p), n, P, _p(m, _f32p), _p(v, _f32p), beta1, beta2, eps,
                               int(step), d, int(seed), bits, _p(codes, _u8p), _p(scales, _f32p),
                               _p(sumsq, _i32p), _p(proj, _f32p))
    return (codes, scales, sumsq, proj) if want_proj else (codes, scales, sumsq)
