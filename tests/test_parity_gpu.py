"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs. Integers, bytes and indices must match bit for bit; floats within the stated
tolerance (projection 1e-3 relative, aggregated scores 1e-5 of sum|eta|)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2502_01703_b200 import binding as B
from paper_2502_01703_b200 import workloads as W

pytestmark = pytest.mark.gpu

DEV = "cuda"
PROJ_TOL = 1e-3
SCORE_TOL = 1e-5


def _np(t):
    return t.detach().cpu().numpy()


def _audit_codes_against_oracle_quantiser(proj, codes, scales, sumsq, bits, max_rows=2):
    """Stage 2 of the GPU path against the oracle's stage 2 on the SAME fp32 projection (the GPU's own). Scales agree
    to the last bits of the norm (reduced in another order, both in fp64). A row's codes may differ from the oracle's
    only through that last bit: every differing code is audited, it must be one level away and alpha * yhat / S must
    lie within 1e-5 of the rounding boundary between the two levels. At 1 bit (a sign) nothing may differ. Rows
    without a differing code have the oracle's code norm. At most `max_rows` rows may need the audit at all."""
    d = proj.shape[1]
    wc, ws, wss = oracle.quantize_rows(proj, bits, normalize=True)
    assert np.allclose(scales, ws, rtol=3e-7, atol=0)
    bad_rows = np.where((codes != wc).any(axis=1))[0]
    assert len(bad_rows) <= max_rows, f"{len(bad_rows)} rows differ from the oracle's codes"
    alpha = 2 ** (bits - 1) - 1 if bits > 1 else 1
    for r in bad_rows:
        assert bits > 1, f"row {r}: sign codes differ"
        qa = oracle.unpack(codes[r], d, bits).astype(np.int32)
        qb = oracle.unpack(wc[r], d, bits).astype(np.int32)
        diff = np.where(qa != qb)[0]
        assert np.abs(qa - qb).max() == 1, f"row {r}: a code differs by more than one level"
        yh = oracle.normalize(proj[r])[0].astype(np.float64)
        pos = alpha * yh[diff] / float(ws[r])
        boundary = (qa[diff] + qb[diff]) / 2.0                  # the half-integer between the two codes
        assert np.all(np.abs(pos - boundary) < 1e-5), f"row {r}: a differing code is not at a rounding boundary"
    if sumsq is not None:
        ok = np.setdiff1d(np.arange(proj.shape[0]), bad_rows)
        assert np.array_equal(sumsq[ok], wss[ok])
    return len(bad_rows)


# ----------------------------------------------------------------------------------------------
# Projection-matrix entries (bit-exact)
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("seed,r0,nr,j0,nj", [
    (0, 0, 8, 0, 256), (0x9E3779B97F4A7C15, 5, 3, 120, 300), (42, 8190, 2, (1 << 23) - 200, 200),
    (7, 0, 1, 0, 1), (7, 100, 130, 64, 129),
])
def test_philox_entries_bit_exact(seed, r0, nr, j0, nj):
    got = _np(B.qless_philox_entries(seed, r0, nr, j0, nj))
    want = oracle.rademacher_rows(seed, r0, nr, j0, nj)
    assert np.array_equal(got, want)


# ----------------------------------------------------------------------------------------------
# Adam prologue (bit-exact bf16)
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("step", [0, 7])
@pytest.mark.parametrize("use_adam", [True, False])
def test_adam_gamma_bit_exact(dtype, step, use_adam):
    n, P = 5, 1024
    g = W.student_t_gradients(n, P, seed=11, device=DEV, dtype=dtype)
    m, v = W.adam_moments(P, seed=12, device=DEV)
    cfg = dict(beta1=0.9, beta2=0.999, eps=1e-8, step=step)
    got = B.qless_adam_gamma(g, m if use_adam else None, v if use_adam else None, cfg)
    g32 = _np(g.float())
    want = oracle.adam_gamma(g32, _np(m) if use_adam else None, _np(v) if use_adam else None, **cfg)
    assert np.array_equal(_np(got.float()).view(np.uint32), want.view(np.uint32))


def test_adam_gamma_bit_exact_on_many_elements():
    # 2^26 elements: the approximate-unit fast path must round to the oracle's bf16 everywhere, also for the few
    # per ten thousand elements that fall next to a rounding boundary and take the exact sequence
    n, P = 64, 1 << 20
    g = W.student_t_gradients(n, P, seed=13, device=DEV, dtype=torch.bfloat16)
    m, v = W.adam_moments(P, seed=14, device=DEV)
    got = _np(B.qless_adam_gamma(g, m, v, dict(beta1=0.9, beta2=0.999, eps=1e-8, step=0)).float())
    want = oracle.adam_gamma(_np(g.float()), _np(m), _np(v))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("v_scale,eps", [(1e-12, 1e-8), (1e-10, 1e-8), (1e-14, 1e-8), (1e-6, 0.0), (1e-6, 1e-3), (1e-30, 1e-8)])
def test_adam_gamma_bit_exact_across_eps_over_sqrt_v(v_scale, eps):
    # eps / sqrt(v') from far below to far above the bound under which the kernel's one-unit fast path is used:
    # both sides of that bound, and the elements next to it, must round to the oracle's bf16
    n, P = 16, 1 << 16
    g = W.student_t_gradients(n, P, seed=15, device=DEV, dtype=torch.bfloat16) * (v_scale ** 0.5 * 30)
    m, v = W.adam_moments(P, seed=16, device=DEV)
    v = v * (v_scale / 1e-6)
    v *= torch.logspace(-2, 2, P, device=DEV)                   # four decades of v across the coordinates
    cfg = dict(beta1=0.9, beta2=0.999, eps=eps, step=0)
    got = _np(B.qless_adam_gamma(g, m, v, cfg).float())
    want = oracle.adam_gamma(_np(g.float()), _np(m), _np(v), **cfg)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_adam_gamma_strided_rows_and_extreme_values():
    n, P = 3, 256
    big = torch.zeros((n, P + 64), dtype=torch.float32, device=DEV)
    g = big[:, :P]
    g.copy_(W.student_t_gradients(n, P, seed=13, device=DEV))
    g[0, 0] = 0.0; g[0, 1] = 1e30; g[0, 2] = -1e-30; g[1, 5] = 3e38
    m, v = W.adam_moments(P, seed=14, device=DEV)
    v[3] = 0.0; m[3] = 0.0
    got = B.qless_adam_gamma(g, m, v)
    want = oracle.adam_gamma(_np(g), _np(m), _np(v))
    assert np.array_equal(_np(got.float()).view(np.uint32), want.view(np.uint32))


# ----------------------------------------------------------------------------------------------
# Normalise + quantise + pack
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("bits", [8, 4, 2, 1])
@pytest.mark.parametrize("d", [128, 512, 8192])
def test_quantize_bit_exact_on_identical_normalised_inputs(bits, d):
    # protocol: rows are normalised by the oracle (Eq. 2), both sides then quantise the same fp32 values
    n = 37
    y = _np(W.student_t_gradients(n, d, seed=20 + bits, device=DEV))
    y[5] = 0.0                                   # zero vector
    yh = np.stack([oracle.normalize(r)[0] for r in y])
    # plant exact rounding ties: alpha * x / S = k + 0.5 for the row whose absmax is made 1.0
    if bits > 1:
        alpha = 2 ** (bits - 1) - 1
        yh[7, :] = 0.0
        yh[7, 0] = 1.0
        for k in range(min(alpha, 20)):
            yh[7, 1 + k] = np.float32((k + 0.5) / alpha) * (1 if k % 2 else -1)
    codes, scales, sumsq = B.qless_quantize(torch.from_numpy(yh).to(DEV), bits, normalize=False)
    wc, ws, wss = oracle.quantize_rows(yh, bits, normalize=False)
    assert np.array_equal(_np(codes), wc)
    assert np.array_equal(_np(scales).view(np.uint32), ws.view(np.uint32))
    assert np.array_equal(_np(sumsq), wss)


@pytest.mark.parametrize("bits", [8, 4, 2, 1])
def test_quantize_with_normalisation_near_tie_audit(bits):
    # With Eq. 2 done on the GPU the norm is reduced in a different order (still in fp64); codes may then
    # differ only where alpha*yhat/S sits within 1e-5 of a rounding boundary, and by one level.
    n, d = 300, 8192
    y = _np(W.student_t_gradients(n, d, seed=30, device=DEV)) * np.float32(1e-3)
    codes, scales, sumsq = B.qless_quantize(torch.from_numpy(y).to(DEV), bits, normalize=True)
    wc, ws, wss = oracle.quantize_rows(y, bits, normalize=True)
    codes, scales = _np(codes), _np(scales)
    assert np.allclose(scales, ws, rtol=3e-7, atol=0)
    bad_rows = np.where((codes != wc).any(axis=1))[0]
    assert len(bad_rows) <= 3, f"{len(bad_rows)} rows differ"
    alpha = 2 ** (bits - 1) - 1 if bits > 1 else 1
    for r in bad_rows:
        qa = oracle.unpack(codes[r], d, bits).astype(np.int32)
        qb = oracle.unpack(wc[r], d, bits).astype(np.int32)
        diff = np.where(qa != qb)[0]
        assert bits > 1 and np.abs(qa - qb).max() == 1
        yh = oracle.normalize(y[r])[0].astype(np.float64)
        pos = alpha * yh[diff] / float(ws[r])
        assert np.all(np.abs(np.abs(pos - np.floor(pos)) - 0.5) < 1e-5)


# Absmean variant: same protocol as above. The mean absolute value is reduced in another order than the oracle's
# (both in fp64), so codes may differ only where yhat / Delta sits within 1e-5 of a rounding boundary, by one level.
@pytest.mark.parametrize("bits", [8, 4, 2, 1])
@pytest.mark.parametrize("normalize", [False, True])
def test_quantize_absmean_matches_oracle(bits, normalize):
    n, d = 200, 8192
    y = _np(W.student_t_gradients(n, d, seed=33, device=DEV)) * np.float32(1e-2)
    y[5] = 0.0
    y[6, :] = np.tile(np.array([0.5, -1.5, 2.0, 0.0], np.float32), d // 4)      # mean |x| = 1: ties and clipping
    codes, scales, sumsq = B.qless_quantize_absmean(torch.from_numpy(y).to(DEV), bits, normalize=normalize)
    wc, ws, wss = oracle.quantize_absmean_rows(y, bits, normalize=normalize)
    codes, scales, sumsq = _np(codes), _np(scales), _np(sumsq)
    assert np.allclose(scales, ws, rtol=3e-7, atol=0)
    if not normalize:
        assert np.array_equal(codes[6], wc[6]) and scales[6] == ws[6]
    bad_rows = np.where((codes != wc).any(axis=1))[0]
    assert len(bad_rows) <= 3, f"{len(bad_rows)} rows differ"
    alpha = 2 ** (bits - 1) - 1 if bits > 1 else 1
    for r in bad_rows:
        qa = oracle.unpack(codes[r], d, bits).astype(np.int32)
        qb = oracle.unpack(wc[r], d, bits).astype(np.int32)
        diff = np.where(qa != qb)[0]
        assert bits > 1 and np.abs(qa - qb).max() == 1
        yh = (oracle.normalize(y[r])[0] if normalize else y[r]).astype(np.float64)
        pos = alpha * yh[diff] / float(ws[r])
        assert np.all(np.abs(np.abs(pos - np.floor(pos)) - 0.5) < 1e-5)
    ok = np.setdiff1d(np.arange(n), bad_rows)
    assert np.array_equal(sumsq[ok], wss[ok])
    # such a store goes through the scorer unchanged
    if bits == 4 and normalize:
        tc = torch.from_numpy(wc[:64].copy()).to(DEV).unsqueeze(0); vc = torch.from_numpy(wc[64:96].copy()).to(DEV).unsqueeze(0)
        ts = torch.from_numpy(ws[:64].copy()).to(DEV).unsqueeze(0); vs = torch.from_numpy(ws[64:96].copy()).to(DEV).unsqueeze(0)
        got = B.qless_score(tc, vc, ts, vs, [1.0], [0, 32], d, bits)
        want = oracle.score(wc[None, :64], wc[None, 64:96], ws[None, :64], ws[None, 64:96], [1.0], [0, 32], d, bits)
        assert np.abs(_np(got) - want).max() <= SCORE_TOL


def test_quantize_edge_shapes():
    for n in (0, 1, 2):
        x = torch.randn((n, 256), device=DEV)
        codes, scales, sumsq = B.qless_quantize(x, 4)
        assert codes.shape == (n, 128) and scales.shape == (n,)
    x = torch.zeros((4, 1024), device=DEV)
    for bits in (8, 4, 2, 1):
        codes, scales, sumsq = B.qless_quantize(x, bits)
        assert not _np(codes).any() and not _np(scales).any() and not _np(sumsq).any()


# ----------------------------------------------------------------------------------------------
# Projection
# ----------------------------------------------------------------------------------------------

def _proj_err(got, want):
    num = np.linalg.norm(got.astype(np.float64) - want.astype(np.float64), axis=1)
    den = np.linalg.norm(want.astype(np.float64), axis=1)
    rel_l2 = (num / den).max()
    rel_max = (np.abs(got - want).max(axis=1) / np.abs(want).max(axis=1)).max()
    return rel_l2, rel_max


@pytest.mark.parametrize("n,P,d,dtype,use_adam", [
    (37, 1024, 256, torch.float32, True),
    (300, 4096, 128, torch.bfloat16, True),
    (5, 2048 + 128, 512, torch.bfloat16, False),
    (1, 128, 128, torch.float32, False),
    (64, 1 << 16, 256, torch.bfloat16, True),
])
def test_projection_matches_oracle(n, P, d, dtype, use_adam):
    seed = 0xC0FFEE
    g = W.student_t_gradients(n, P, seed=40, device=DEV, dtype=dtype)
    m, v = W.adam_moments(P, seed=41, device=DEV)
    out = B.qless_project_quantize(g, d, seed, 8, m if use_adam else None, v if use_adam else None, want_proj=True)
    gamma = oracle.adam_gamma(_np(g.float()), _np(m) if use_adam else None, _np(v) if use_adam else None)
    want = oracle.project(gamma, d, seed)
    rel_l2, rel_max = _proj_err(_np(out["proj"]), want)
    assert rel_l2 <= PROJ_TOL and rel_max <= PROJ_TOL, (rel_l2, rel_max)
    # downstream of the GPU's own projection the integer stages are exact: oracle quantiser on proj_out (a row
    # may sit on a rounding tie through the norm's last bit: audited code by code)
    _audit_codes_against_oracle_quantiser(_np(out["proj"]), _np(out["codes"]), _np(out["scales"]), _np(out["sumsq"]), 8, max_rows=1)


def test_projection_of_basis_vectors_is_exact():
    # e_j projects to column j of R: entries exactly +-1/sqrt(d), unit norm
    P, d, seed = 1024, 256, 77
    js = [0, 1, 127, 128, 1023]
    g = torch.zeros((len(js), P), dtype=torch.bfloat16, device=DEV)
    for a, j in enumerate(js):
        g[a, j] = 1.0
    out = B.qless_project_quantize(g, d, seed, 1, want_proj=True)
    proj = _np(out["proj"])
    for a, j in enumerate(js):
        col = oracle.rademacher_rows(seed, 0, d, j, 1)[:, 0].astype(np.float32)
        assert np.array_equal(proj[a], col * np.float32(1.0 / np.sqrt(np.float32(d))))
        assert np.array_equal(oracle.unpack(_np(out["codes"])[a], d, 1), col.astype(np.int8))


def test_projection_is_deterministic_and_handles_empty_batch():
    g = W.student_t_gradients(70, 8192, seed=43, device=DEV, dtype=torch.bfloat16)
    a = B.qless_project_quantize(g, 512, 3, 4, want_proj=True)
    b = B.qless_project_quantize(g, 512, 3, 4, want_proj=True)
    assert torch.equal(a["proj"], b["proj"]) and torch.equal(a["codes"], b["codes"])
    e = B.qless_project_quantize(g[:0], 512, 3, 4)
    assert e["codes"].shape == (0, 256)


# ----------------------------------------------------------------------------------------------
# Gaussian projection matrix (the other distribution Sec. 2.4 allows for R)
# ----------------------------------------------------------------------------------------------

@pytest.fixture
def restore_projection_path():
    try:
        yield
    finally:
        B.qless_set_projection_path(0)


@pytest.mark.parametrize("seed,r0,nr,j0,nj", [
    (0, 0, 8, 0, 512), (0x9E3779B97F4A7C15, 5, 3, 120, 301), (42, 8190, 2, (1 << 23) - 200, 200),
    (7, 0, 1, 4, 1), (7, 100, 130, 64, 130), (3, 1, 2, (1 << 36) + 8, 64),
])
def test_gaussian_entries_match_oracle(seed, r0, nr, j0, nj):
    # The device evaluates ln, sqrt, sin and cos in fp32, the oracle in fp64: an entry may land on the other side
    # of a bf16 rounding boundary. Such entries must be rare and differ by exactly one bf16 step; all others are
    # bit-identical.
    got = _np(B.qless_gaussian_entries(seed, r0, nr, j0, nj))
    want = oracle.gaussian_rows(seed, r0, nr, j0, nj)
    gb = (got.view(np.uint32) >> 16).astype(np.int64)
    wb = (want.view(np.uint32) >> 16).astype(np.int64)
    assert np.all((got.view(np.uint32) & 0xFFFF) == 0)          # bf16-representable
    diff = np.abs(gb - wb)
    assert diff.max() <= 1
    assert (diff != 0).sum() <= max(1, int(2e-3 * got.size)), (int((diff != 0).sum()), got.size)


@pytest.mark.parametrize("n,P,d,dtype,use_adam", [
    (37, 1024, 256, torch.float32, True),
    (300, 4096, 128, torch.bfloat16, True),
    (5, 2048 + 128, 512, torch.bfloat16, False),
    (64, 1 << 16, 256, torch.bfloat16, True),
])
def test_gaussian_projection_matches_oracle(restore_projection_path, n, P, d, dtype, use_adam):
    seed = 0xBADC0DE
    g = W.student_t_gradients(n, P, seed=44, device=DEV, dtype=dtype)
    m, v = W.adam_moments(P, seed=45, device=DEV)
    out = B.qless_project_quantize(g, d, seed, 4, m if use_adam else None, v if use_adam else None, want_proj=True, matrix=B.GAUSSIAN)
    B.qless_check()
    gamma = oracle.adam_gamma(_np(g.float()), _np(m) if use_adam else None, _np(v) if use_adam else None)
    want = oracle.project_gaussian(gamma, d, seed)
    rel_l2, rel_max = _proj_err(_np(out["proj"]), want)
    assert rel_l2 <= PROJ_TOL and rel_max <= PROJ_TOL, (rel_l2, rel_max)
    # the integer stages downstream are the same kernels: oracle quantiser on the GPU's own projection
    _audit_codes_against_oracle_quantiser(_np(out["proj"]), _np(out["codes"]), _np(out["scales"]), _np(out["sumsq"]), 4, max_rows=1)
    # the CUDA-core kernel generates the same entries: only the fp32 summation order differs
    B.qless_set_projection_path(1)
    ref = B.qless_project_quantize(g, d, seed, 4, m if use_adam else None, v if use_adam else None, want_proj=True, matrix=B.GAUSSIAN)
    e_l2, e_max = _proj_err(_np(out["proj"]), _np(ref["proj"]))
    assert e_l2 <= 1e-5 and e_max <= 1e-5, (e_l2, e_max)


def test_gaussian_projection_full_width_sampled():
    # config 5's gradient width (P = 2^22, bf16, Adam), a full 256-row batch, d = 8192: the launch configuration of
    # the large runs (64 K chunks, every CTA pair persistent); the oracle evaluates sampled rows and coordinates
    n, P, d, seed = 256, 1 << 22, 8192, 4242
    g = W.student_t_gradients(n, P, seed=46, device=DEV, dtype=torch.bfloat16)
    m, v = W.adam_moments(P, seed=47, device=DEV)
    out = B.qless_project_quantize(g, d, seed, 2, m, v, want_proj=True, matrix=B.GAUSSIAN)
    B.qless_check()
    rows, coords = [0, 130, 255], [0, 129, 4096, 8191]
    gamma = oracle.adam_gamma(_np(g[rows].float()), _np(m), _np(v)).astype(np.float64)
    proj = _np(out["proj"])
    ref = np.abs(proj[rows]).max(axis=1)
    for b, r in enumerate(coords):
        z = oracle.gaussian_rows(seed, r, 1, 0, P)[0].astype(np.float64)
        want = (gamma @ z) * float(np.float32(1.0) / np.sqrt(np.float32(d)))
        assert (np.abs(proj[rows, r] - want) / ref).max() <= PROJ_TOL
    # JL for a Gaussian matrix: ||y||^2 / ||Gamma||^2 within 5 sigma of 1
    g2 = (gamma ** 2).sum(1)
    y2 = (proj[rows].astype(np.float64) ** 2).sum(1)
    assert np.all(np.abs(y2 / g2 - 1) <= 5 * math.sqrt(2.0 / d))


def test_gaussian_host_entry_matches_device_entry():
    # the host-buffer entry projects column slabs with the Philox counters offset by the slab's first column: with
    # the Gaussian matrix, too, it must give the device-buffer entry's bytes
    n, P, d, bits = 70, 1 << 18, 256, 4
    g = W.student_t_gradients(n, P, seed=63, device="cpu").to(torch.bfloat16)
    host = g.clone().pin_memory()
    m, v = W.adam_moments(P, seed=64, device=DEV)
    dev_out = B.qless_project_quantize(g.to(DEV), d, 778, bits, adam_m=m, adam_v=v, matrix=B.GAUSSIAN)
    host_out = B.qless_project_quantize_host(host, d, 778, bits, adam_m=m, adam_v=v, device=DEV, matrix=B.GAUSSIAN)
    torch.cuda.synchronize()
    assert np.array_equal(host_out["codes"].numpy(), _np(dev_out["codes"]))
    assert np.array_equal(host_out["scales"].numpy(), _np(dev_out["scales"]))
    # and it is not the Rademacher result, which the plain call and an explicit RADEMACHER both give
    rad = B.qless_project_quantize(g.to(DEV), d, 778, bits, adam_m=m, adam_v=v)
    rad2 = B.qless_project_quantize(g.to(DEV), d, 778, bits, adam_m=m, adam_v=v, matrix=B.RADEMACHER)
    assert torch.equal(rad["codes"], rad2["codes"])
    assert not np.array_equal(_np(rad["codes"]), _np(dev_out["codes"]))


def test_gaussian_projection_of_basis_vectors():
    # e_j projects to column j of the matrix the entry hook returns, scaled by the fp32 value of 1/sqrt(d)
    P, d, seed = 1024, 256, 78
    js = [0, 1, 2, 3, 127, 128, 1023]
    g = torch.zeros((len(js), P), dtype=torch.bfloat16, device=DEV)
    for a, j in enumerate(js):
        g[a, j] = 1.0
    proj = _np(B.qless_project_quantize(g, d, seed, 8, want_proj=True, matrix=B.GAUSSIAN)["proj"])
    for a, j in enumerate(js):
        col = _np(B.qless_gaussian_entries(seed, 0, d, j - j % 4, 4))[:, j % 4]
        assert np.array_equal(proj[a], col * np.float32(1.0 / np.sqrt(np.float32(d))))
    # the matrix is an argument, not a state: the next plain call uses the Rademacher matrix
    proj = _np(B.qless_project_quantize(g, d, seed, 8, want_proj=True)["proj"])
    col = oracle.rademacher_rows(seed, 0, d, 0, 1)[:, 0].astype(np.float32)
    assert np.array_equal(proj[0], col * np.float32(1.0 / np.sqrt(np.float32(d))))
    with pytest.raises(B.QlessError):
        B.qless_project_quantize(g, d, seed, 8, matrix=2)


# ----------------------------------------------------------------------------------------------
# Integer similarity and aggregated scores
# ----------------------------------------------------------------------------------------------

def _make_store(bits, C, N, V, d, seed):
    xt = W.lowrank_gaussian_features(N, d, C, seed=seed, device=DEV)
    xv = W.lowrank_gaussian_features(V, d, C, seed=seed + 1, device=DEV)
    tc = torch.empty((C, N, d * bits // 8), dtype=torch.uint8, device=DEV)
    vc = torch.empty((C, V, d * bits // 8), dtype=torch.uint8, device=DEV)
    ts = torch.empty((C, N), dtype=torch.float32, device=DEV); tss = torch.empty((C, N), dtype=torch.int32, device=DEV)
    vs = torch.empty((C, V), dtype=torch.float32, device=DEV); vss = torch.empty((C, V), dtype=torch.int32, device=DEV)
    for i in range(C):
        c, s, q = B.qless_quantize(xt[i], bits); tc[i] = c; ts[i] = s; tss[i] = q
        c, s, q = B.qless_quantize(xv[i], bits); vc[i] = c; vs[i] = s; vss[i] = q
    return tc, vc, ts, vs, tss, vss


@pytest.mark.parametrize("bits", [8, 4, 2, 1])
@pytest.mark.parametrize("N,V,d", [(150, 70, 256), (65, 129, 1024), (3, 1, 128), (200, 448, 8192)])
def test_score_dots_bit_exact(bits, N, V, d):
    tc, vc, *_ = _make_store(bits, 1, N, V, d, seed=50)
    got = _np(B.qless_score_dots(tc[0], vc[0], d, bits))
    want = oracle.dots(_np(tc[0]), _np(vc[0]), d, bits)
    assert np.array_equal(got, want)
    if N > 10:
        got = _np(B.qless_score_dots(tc[0], vc[0], d, bits, t0=7, nt=3))
        assert np.array_equal(got, want[7:10])


@pytest.mark.parametrize("bits", [8, 4, 2, 1])
@pytest.mark.parametrize("N,V,d", [(300, 449, 8192), (77, 33, 384)])
def test_score_dots_of_arbitrary_code_bytes(bits, N, V, d):
    # every bit pattern is a code: the most negative value of each width (-2 at 2 bits, which the quantiser never emits
    # and the e2m1 operand path has to map to its own -2), d not a multiple of the 256-code K block, two validation tiles
    gen = torch.Generator(device=DEV); gen.manual_seed(77 + bits)
    tc = torch.randint(0, 256, (N, d * bits // 8), generator=gen, device=DEV, dtype=torch.uint8)
    vc = torch.randint(0, 256, (V, d * bits // 8), generator=gen, device=DEV, dtype=torch.uint8)
    got = _np(B.qless_score_dots(tc, vc, d, bits))
    want = oracle.dots(_np(tc), _np(vc), d, bits)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("bits", [8, 4, 2, 1])
@pytest.mark.parametrize("mode", [B.COSINE, B.DEQUANT])
def test_scores_match_oracle(bits, mode):
    C, N, V, d = 3, 333, 100, 512
    eta = [1.0, 0.75, 0.5]
    off = [0, 10, 37, 100]
    tc, vc, ts, vs, tss, vss = _make_store(bits, C, N, V, d, seed=60)
    ts[1, 4] = 0.0; tc[1, 4] = 0; tss[1, 4] = 0          # a zero vector in the store
    got, got_pt = B.qless_score(tc, vc, ts, vs, eta, off, d, bits, train_sumsq=tss, val_sumsq=vss,
                                mode=mode, want_per_task=True)
    want, want_pt = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits, mode=mode, want_per_task=True)
    scale = sum(abs(e) for e in eta) * (1.0 if mode == B.COSINE else max(1e-30, float(np.abs(want_pt).max())))
    assert np.abs(_np(got) - want).max() <= SCORE_TOL * scale
    assert np.abs(_np(got_pt) - want_pt).max() <= SCORE_TOL * scale
    # sumsq recomputed inside the library gives the same scores
    got2 = B.qless_score(tc, vc, ts, vs, eta, off, d, bits, mode=mode)
    assert torch.equal(got2, got)


# More validation vectors than one accumulator tile holds (512 at 8 bits, 448 at the sub-byte widths): the kernel walks
# several validation tiles per train tile, finds the task that each tile starts in and carries a task that straddles
# two tiles in its running sum. Task boundaries are placed across 448 and 512 and off every multiple of 32.
@pytest.mark.parametrize("bits", [8, 4, 2, 1])
@pytest.mark.parametrize("V,off", [(600, [0, 100, 470, 600]), (1100, [0, 100, 470, 530, 1000, 1100]),
                                   (1024, [0, 448, 512, 1024]), (449, [0, 449])])
def test_scores_with_several_validation_tiles(bits, V, off):
    C, N, d = 2, 300, 256
    eta = [1.0, 0.5]
    tc, vc, ts, vs, tss, vss = _make_store(bits, C, N, V, d, seed=160 + V)
    got, got_pt = B.qless_score(tc, vc, ts, vs, eta, off, d, bits, train_sumsq=tss, val_sumsq=vss, want_per_task=True)
    B.qless_check()
    want, want_pt = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits, want_per_task=True)
    assert np.abs(_np(got) - want).max() <= SCORE_TOL * sum(eta)
    assert np.abs(_np(got_pt) - want_pt).max() <= SCORE_TOL * sum(eta)
    # the integer numerators of every tile, bit for bit
    dots = _np(B.qless_score_dots(tc[0], vc[0], d, bits))
    assert np.array_equal(dots, oracle.dots(_np(tc[0]), _np(vc[0]), d, bits))


# 7 and 8 tasks: the tensor-core kernels with one epilogue group (two groups exchange six per-task sums). More tasks
# than the tensor-core epilogue keeps in registers (8): the call takes the CUDA-core kernel.
@pytest.mark.parametrize("bits", [8, 4, 2, 1])
@pytest.mark.parametrize("T", [7, 8, 9, 64])
def test_scores_with_many_tasks(bits, T):
    C, N, V, d = 2, 200, 5 * T + 3, 256
    eta = [1.0, 0.25]
    sizes = [5] * (T - 1) + [8]
    off = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    tc, vc, ts, vs, tss, vss = _make_store(bits, C, N, V, d, seed=170 + T)
    got, got_pt = B.qless_score(tc, vc, ts, vs, eta, off, d, bits, train_sumsq=tss, val_sumsq=vss, want_per_task=True)
    want, want_pt = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits, want_per_task=True)
    assert np.abs(_np(got) - want).max() <= SCORE_TOL * sum(eta)
    assert np.abs(_np(got_pt) - want_pt).max() <= SCORE_TOL * sum(eta)
    # T = 8 is the last count the tensor-core kernel takes: same store, the first eight tasks
    if T == 9:
        off8 = off[:8] + [V]
        got8 = B.qless_score(tc, vc, ts, vs, eta, off8, d, bits)
        want8 = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off8, d, bits)
        assert np.abs(_np(got8) - want8).max() <= SCORE_TOL * sum(eta)


# The CUDA-core kernels (dp4a for 8/4/2-bit codes, XOR + population count for 1-bit codes) stay in the library as
# a second implementation of the same integer similarity: they must agree with the oracle as the tensor-core
# kernel does, and with the tensor-core kernel bit for bit on the raw dots.
@pytest.mark.parametrize("bits", [8, 4, 2, 1])
def test_score_cuda_core_path(bits):
    C, N, V, d = 2, 300, 200, 1024
    eta, off = [1.0, 0.5], [0, 50, 200]
    tc, vc, ts, vs, tss, vss = _make_store(bits, C, N, V, d, seed=65)
    dots_tc = _np(B.qless_score_dots(tc[0], vc[0], d, bits))
    scores_tc = _np(B.qless_score(tc, vc, ts, vs, eta, off, d, bits))
    try:
        B.qless_set_score_path(1)
        dots_cc = _np(B.qless_score_dots(tc[0], vc[0], d, bits))
        scores_cc = _np(B.qless_score(tc, vc, ts, vs, eta, off, d, bits))
    finally:
        B.qless_set_score_path(0)
    want_dots = oracle.dots(_np(tc[0]), _np(vc[0]), d, bits)
    assert np.array_equal(dots_cc, want_dots) and np.array_equal(dots_tc, want_dots)
    want = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits)
    assert np.abs(scores_cc - want).max() <= SCORE_TOL * sum(eta)
    assert np.abs(scores_tc - want).max() <= SCORE_TOL * sum(eta)


# 16-bit baseline (Eq. 3): bf16 rows, fp32 accumulation on the tensor cores against the fp64 definition. Tolerance:
# d products of bf16 values are exact in fp32; their fp32 sum over d = 8192 terms carries a relative error of a few
# 2^-24 sqrt(d) of the norm product in practice (bound d 2^-24), so 2e-5 per unit of |eta| is the stated bar.
SCORE16_TOL = 2e-5

@pytest.mark.parametrize("C,N,V,d,off", [(2, 300, 100, 512, [0, 10, 37, 100]), (1, 65, 129, 128, [0, 129]),
                                         (3, 700, 448, 8192, [0, 150, 300, 448]), (1, 5, 600, 1024, [0, 512, 600])])
def test_score_16bit_matches_oracle(C, N, V, d, off):
    gen = torch.Generator(device=DEV); gen.manual_seed(66 + N)
    tr = torch.randn((C, N, d), generator=gen, device=DEV).to(torch.bfloat16)
    va = torch.randn((C, V, d), generator=gen, device=DEV).to(torch.bfloat16)
    tr[0, 3] = 0                                        # a zero row in the store
    tr[0, 4] = va[0, 1] * 2                             # a row parallel to a validation row
    eta = [1.0, 0.75, 0.5][:C]
    got, got_pt = B.qless_score_16bit(tr, va, eta, off, want_per_task=True)
    want, want_pt = oracle.score_16bit(_np(tr.float()), _np(va.float()), eta, off, want_per_task=True)
    assert np.abs(_np(got) - want).max() <= SCORE16_TOL * sum(eta)
    assert np.abs(_np(got_pt) - want_pt).max() <= SCORE16_TOL * sum(eta)
    assert np.all(_np(got_pt)[3] == 0.0) if C == 1 else True
    # norms kept beside the store give the same scores
    got2 = B.qless_score_16bit(tr, va, eta, off, train_inv_norms=B.qless_inv_norms_16bit(tr), val_inv_norms=B.qless_inv_norms_16bit(va))
    assert torch.equal(got2, got)


# Un-normalised (TracIn-style, Sec. 2.1) scores need no kernel of their own: rows quantised without Eq. 2 keep their
# length in the scale, and the DEQUANT mode sums eta <S_t q_t / alpha, S_v q_v / alpha>. Checked against the oracle on the
# same codes (1e-5 relative) and against the fp64 inner products of the rows themselves (8-bit quantisation error).
def test_unnormalised_scores_through_dequant_mode():
    C, N, V, d, bits = 2, 200, 64, 1024, 8
    gen = torch.Generator(device=DEV); gen.manual_seed(68)
    lens_t = torch.rand((C, N, 1), generator=gen, device=DEV) * 4 + 0.25
    lens_v = torch.rand((C, V, 1), generator=gen, device=DEV) * 2 + 0.5
    xt = torch.randn((C, N, d), generator=gen, device=DEV) * lens_t / np.sqrt(d)
    xv = torch.randn((C, V, d), generator=gen, device=DEV) * lens_v / np.sqrt(d)
    xv = xv + 0.5 * xt[:, :V]                                  # correlated, so that scores are not all near zero
    tc = torch.empty((C, N, d), dtype=torch.uint8, device=DEV); vc = torch.empty((C, V, d), dtype=torch.uint8, device=DEV)
    ts = torch.empty((C, N), device=DEV); vs = torch.empty((C, V), device=DEV)
    for i in range(C):
        tc[i], ts[i], _ = B.qless_quantize(xt[i], bits, normalize=False)
        vc[i], vs[i], _ = B.qless_quantize(xv[i], bits, normalize=False)
    eta, off = [1.0, 0.5], [0, 20, 64]
    got, got_pt = B.qless_score(tc, vc, ts, vs, eta, off, d, bits, mode=B.DEQUANT, want_per_task=True)
    want, want_pt = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits, mode=B.DEQUANT, want_per_task=True)
    scale = float(np.abs(want_pt).max())
    assert np.abs(_np(got_pt) - want_pt).max() <= SCORE_TOL * sum(eta) * scale
    exact = np.zeros((N, 2))
    for i in range(C):
        ip = _np(xt[i]).astype(np.float64) @ _np(xv[i]).astype(np.float64).T
        for j in range(2):
            exact[:, j] += eta[i] * ip[:, off[j]:off[j + 1]].mean(axis=1)
    assert np.abs(_np(got_pt) - exact).max() <= 0.02 * np.abs(exact).max()
    assert np.abs(_np(got) - exact.max(axis=1)).max() <= 0.02 * np.abs(exact).max()


def test_scores_edge_shapes():
    for (C, N, V, T) in [(1, 1, 1, 1), (2, 64, 128, 1), (1, 65, 129, 2), (4, 10, 448, 3)]:
        d, bits = 256, 4
        tc, vc, ts, vs, tss, vss = _make_store(bits, C, N, V, d, seed=70)
        off = [0, V] if T == 1 else ([0, V // 2, V] if T == 2 else [0, 64, 192, 448])
        eta = [1.0, 0.75, 0.5, 0.25][:C]
        got = B.qless_score(tc, vc, ts, vs, eta, off, d, bits)
        want = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits)
        assert np.abs(_np(got) - want).max() <= SCORE_TOL * sum(eta)
    # N = 0
    tc, vc, ts, vs, _, _ = _make_store(8, 1, 4, 4, 128, seed=71)
    assert B.qless_score(tc[:, :0], vc, ts[:, :0], vs, [1.0], [0, 4], 128, 8).numel() == 0


# ----------------------------------------------------------------------------------------------
# Host-buffer entry: the batch is copied in column slabs that overlap the projection of earlier slabs;
# codes, scales and code norms must be those of the device-buffer entry, bit for bit.
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n,P,d,bits,dtype,adam", [
    (40, 32768, 256, 4, torch.bfloat16, True),       # 32 K chunks -> 8 slabs of 4
    (33, 4736, 128, 8, torch.float32, False),        # 5 chunks, the last one ragged -> 5 slabs
    (5, 1024, 512, 1, torch.float32, True),          # a single chunk -> one slab
    (300, 65536, 1024, 2, torch.bfloat16, True),     # two gradient-row tiles
])
def test_host_entry_matches_device_entry(n, P, d, bits, dtype, adam):
    g = W.student_t_gradients(n, P, seed=61 + n, device="cpu").to(dtype)
    pitch = P + 64                                            # rows of the host buffer need not be contiguous
    host = torch.zeros((n, pitch), dtype=dtype).pin_memory()
    host[:, :P] = g
    m = v = cfg = None
    if adam:
        m, v = W.adam_moments(P, seed=62, device=DEV)
        cfg = dict(beta1=0.9, beta2=0.999, eps=1e-8, step=0)
    dev_out = B.qless_project_quantize(g.to(DEV), d, 777, bits, adam_m=m, adam_v=v, adam=cfg)
    for rep in range(2):                                      # the second call reuses the staging buffers
        host_out = B.qless_project_quantize_host(host[:, :P], d, 777, bits, adam_m=m, adam_v=v, adam=cfg, device=DEV)
        torch.cuda.synchronize()
        assert np.array_equal(host_out["codes"].numpy(), _np(dev_out["codes"]))
        assert np.array_equal(host_out["scales"].numpy(), _np(dev_out["scales"]))
        assert np.array_equal(host_out["sumsq"].numpy(), _np(dev_out["sumsq"]))


# ----------------------------------------------------------------------------------------------
# Top-k (bit-exact index sets, ascending order)
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("N", [1, 2, 7, 8, 9, 63, 1000, 2048, 2049, 100_003, 270_000, 360_448, 360_449, 1 << 21])
@pytest.mark.parametrize("frac", [0.0, 0.01, 0.05, 0.5, 1.0])
def test_topk_matches_oracle(N, frac):
    gen = torch.Generator(device=DEV); gen.manual_seed(80 + N)
    s = torch.randn(N, generator=gen, device=DEV)
    got = _np(B.qless_select_topk(s, frac))
    want = oracle.select_topk(_np(s), frac)
    assert np.array_equal(got, want)
    # up to 360 448 scores the default is the one-launch cluster kernel; the multi-pass kernels must agree with it
    try:
        B.qless_set_select_path(1)
        assert np.array_equal(_np(B.qless_select_topk(s, frac)), want)
    finally:
        B.qless_set_select_path(0)


def test_topk_ties_and_special_values():
    gen = torch.Generator(device=DEV); gen.manual_seed(90)
    N = 50_000
    s = torch.round(torch.randn(N, generator=gen, device=DEV) * 4) / 4     # heavy ties
    s[100] = float("inf"); s[200] = float("-inf"); s[300] = float("nan"); s[400] = -0.0; s[401] = 0.0
    for frac in (0.001, 0.05, 0.3, 0.9, 1.0):
        assert np.array_equal(_np(B.qless_select_topk(s, frac)), oracle.select_topk(_np(s), frac))
    c = torch.full((7777,), 2.5, device=DEV)
    assert np.array_equal(_np(B.qless_select_topk(c, 0.1)), np.arange(777))
    z = torch.tensor([0.0, -0.0, 0.0, -0.0], device=DEV)
    assert _np(B.qless_select_topk(z, 0.5)).tolist() == [0, 2]
    q = torch.tensor([float("nan"), float("-inf"), 1.0, float("inf")], device=DEV)
    assert _np(B.qless_select_topk(q, 0.75)).tolist() == [1, 2, 3]


def _large_scores(kind, N, seed):
    gen = torch.Generator(device=DEV); gen.manual_seed(seed)
    if kind == "gauss":
        return torch.randn(N, generator=gen, device=DEV)
    if kind == "ties":
        return torch.round(torch.randn(N, generator=gen, device=DEV) * 8) / 8
    if kind == "const":
        return torch.full((N,), -1.25, device=DEV)
    if kind == "ascending":
        return torch.arange(N, device=DEV, dtype=torch.float32) * (1.0 / 1024)
    if kind == "descending":
        return -torch.arange(N, device=DEV, dtype=torch.float32) * (1.0 / 1024)
    if kind == "spike":       # almost all scores equal, a few thousand larger ones packed into one stretch
        s = torch.zeros(N, device=DEV)
        s[N // 3: N // 3 + 5000] = torch.rand(5000, generator=gen, device=DEV) + 1.0
        return s
    raise ValueError(kind)


# Above 2^22 scores the selection brackets the k-th largest key from a sample, gathers the candidates
# in one pass and selects among them; the three paths must return the oracle's set, in order.
@pytest.mark.parametrize("kind,N", [("gauss", (1 << 22) + 1), ("gauss", 5_000_003), ("ties", 6_000_000),
                                     ("const", (1 << 22) + 4097), ("ascending", 4_500_000),
                                     ("descending", 4_500_001), ("spike", 5_000_000), ("gauss", (1 << 24) + 77)])
def test_topk_large_bracketed(kind, N):
    s = _large_scores(kind, N, 95 + N % 1000)
    s_np = _np(s)
    for frac in (1e-6, 0.0005, 0.05, 0.5, 1.0):
        want = oracle.select_topk(s_np, frac)
        got = _np(B.qless_select_topk(s, frac))
        assert got.shape == want.shape and np.array_equal(got, want), (kind, N, frac)
    try:
        for path in (1, 2):
            B.qless_set_select_path(path)
            got = _np(B.qless_select_topk(s, 0.05))
            assert np.array_equal(got, oracle.select_topk(s_np, 0.05)), (kind, N, path)
    finally:
        B.qless_set_select_path(0)


# At 2^28 scores (the size at which the selection is timed against HBM bandwidth) the oracle's sort is out of
# reach of a test, so the result is checked through what defines it: k indices, strictly ascending, and no
# unselected score above the smallest selected one (ties at the threshold: the smallest indices are taken).
def test_topk_2pow28_properties():
    N, frac = 1 << 28, 0.05
    gen = torch.Generator(device=DEV); gen.manual_seed(97)
    s = torch.randn(N, generator=gen, device=DEV)
    s[12345] = float("nan"); s[N - 1] = float("inf"); s[7] = float("-inf")
    idx = B.qless_select_topk(s, frac)
    k = int(np.floor(frac * N + 1e-6))
    assert idx.numel() == k
    assert bool((idx[1:] > idx[:-1]).all()) and int(idx[0]) >= 0 and int(idx[-1]) == N - 1
    sel = torch.zeros(N, dtype=torch.bool, device=DEV)
    sel[idx] = True
    assert not bool(sel[12345]) and not bool(sel[7])
    thr = s[idx].min()
    rest = torch.where(sel | torch.isnan(s), torch.full_like(s, float("-inf")), s)
    top_rest = rest.max()
    assert float(top_rest) <= float(thr)
    if float(top_rest) == float(thr):        # ties at the threshold: every unselected tie lies after every selected one
        tie_sel = torch.nonzero(sel & (s == thr)).max()
        tie_uns = torch.nonzero(~sel & (s == thr)).min()
        assert int(tie_uns) > int(tie_sel)
    del sel, rest


# ----------------------------------------------------------------------------------------------
# Config 1: tiny end to end (1000 train + 64 val, P = 8192 fp32, d = 512, 8-bit, 2 checkpoints,
# lr [1, 0.5], 2 tasks of 32, top 5 %)
# ----------------------------------------------------------------------------------------------

def _audit_codes_of_two_pipelines(codes_gpu, codes_or, proj_or, eps, bits):
    """Codes of the GPU pipeline against codes of the oracle's own pipeline (different fp32 / fp64 projections).
    alpha * yhat_m / S = alpha * y_m / max|y| does not depend on the norm, and a projection error of at most eps
    (relative to max|y|, as measured for this batch) moves it by at most 2 alpha eps (the element and the maximum each
    move by eps max|y|). So a code may differ from the oracle's only by one level and only where the oracle's own
    position lies within 2 alpha eps (+ 1e-6 for the fp32 steps of both quantisers) of the boundary between the two
    levels; at 1 bit only where |y_m| <= eps max|y|. Returns the number of differing codes per row."""
    d = proj_or.shape[1]
    alpha = 2 ** (bits - 1) - 1 if bits > 1 else 1
    flips = np.zeros(codes_gpu.shape[0], np.int64)
    for r in np.where((codes_gpu != codes_or).any(axis=1))[0]:
        qa = oracle.unpack(codes_gpu[r], d, bits).astype(np.int32)
        qb = oracle.unpack(codes_or[r], d, bits).astype(np.int32)
        diff = np.where(qa != qb)[0]
        flips[r] = diff.size
        y = proj_or[r].astype(np.float64)
        ymax = np.abs(y).max()
        if bits == 1:
            assert np.all(np.abs(y[diff]) <= eps * ymax * (1 + 1e-6))
        else:
            assert np.abs(qa - qb).max() == 1
            pos = alpha * y[diff] / ymax
            assert np.all(np.abs(pos - (qa[diff] + qb[diff]) / 2.0) <= 2 * alpha * eps + 1e-6)
    return flips


@pytest.mark.parametrize("bits", [8, 1])
def test_config1_end_to_end(bits):
    cfg = W.CONFIGS["c1_tiny_e2e"]
    P, d, C, seed = cfg["P"], cfg["d"], cfg["C"], 2025
    nt, nv = cfg["n_train"], cfg["n_val"]
    off = _np(W.task_offsets(cfg["tasks"])).tolist()
    rb = d * bits // 8
    tc = torch.empty((C, nt, rb), dtype=torch.uint8, device=DEV); vc = torch.empty((C, nv, rb), dtype=torch.uint8, device=DEV)
    ts = torch.empty((C, nt), device=DEV); vs = torch.empty((C, nv), device=DEV)
    tss = torch.empty((C, nt), dtype=torch.int32, device=DEV); vss = torch.empty((C, nv), dtype=torch.int32, device=DEV)
    o_tc = np.empty((C, nt, rb), np.uint8); o_vc = np.empty((C, nv, rb), np.uint8)
    o_ts = np.empty((C, nt), np.float32); o_vs = np.empty((C, nv), np.float32)
    flips_t = np.zeros((C, nt), np.int64); flips_v = np.zeros((C, nv), np.int64)
    for i in range(C):
        g_tr = W.student_t_gradients(nt, P, seed=100 + i, device=DEV)
        g_va = W.student_t_gradients(nv, P, seed=200 + i, device=DEV)
        m, v = W.adam_moments(P, seed=300 + i, device=DEV)
        a = B.qless_project_quantize(g_tr, d, seed, bits, m, v, want_proj=True)
        b = B.qless_project_quantize(g_va, d, seed, bits, want_proj=True)
        tc[i], ts[i], tss[i] = a["codes"], a["scales"], a["sumsq"]
        vc[i], vs[i], vss[i] = b["codes"], b["scales"], b["sumsq"]
        # oracle, stage by stage
        for out, g, mv, o_codes, o_scales, flips in ((a, g_tr, (_np(m), _np(v)), o_tc, o_ts, flips_t),
                                                     (b, g_va, (None, None), o_vc, o_vs, flips_v)):
            oc, os_, _, op = oracle.project_quantize(_np(g), d, seed, bits, m=mv[0], v=mv[1], want_proj=True)
            rel_l2, rel_max = _proj_err(_np(out["proj"]), op)
            assert rel_l2 <= PROJ_TOL and rel_max <= PROJ_TOL
            o_codes[i], o_scales[i] = oc, os_
            # stage 2 on the GPU's own projection: the oracle's codes up to the audited last-bit ties
            _audit_codes_against_oracle_quantiser(_np(out["proj"]), _np(out["codes"]), _np(out["scales"]), _np(out["sumsq"]), bits)
            # the two pipelines' codes: they differ only where the measured projection error allows it
            flips[i] = _audit_codes_of_two_pipelines(_np(out["codes"]), oc, op, rel_max, bits)
    eta = cfg["lr"]
    scores = B.qless_score(tc, vc, ts, vs, eta, off, d, bits, train_sumsq=tss, val_sumsq=vss)
    # (a) same codes in, same scores out
    want_same = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits)
    assert np.abs(_np(scores) - want_same).max() <= SCORE_TOL * sum(eta)
    idx = _np(B.qless_select_topk(scores, cfg["frac"]))
    assert idx.size == 50
    assert np.array_equal(idx, oracle.select_topk(_np(scores), cfg["frac"]))     # bit-exact given the same scores
    # (b) whole pipeline against the oracle's own pipeline. The bar follows from the code differences counted above:
    # a code vector q with f codes moved by one level (by two, at 1 bit: -1 <-> +1) turns by an angle of at most
    # asin(step sqrt(f) / ||q||), and a cosine moves by at most the sum of the angles its two vectors turn by
    # (triangle inequality on the sphere). Summed with |eta| and with the worst validation vector of each checkpoint:
    step = 2.0 if bits == 1 else 1.0
    nrm_t = np.sqrt(_np(tss).astype(np.float64)); nrm_v = np.sqrt(_np(vss).astype(np.float64))
    ang_t = np.arcsin(np.minimum(1.0, step * np.sqrt(flips_t) / np.maximum(nrm_t - step * np.sqrt(flips_t), 1.0)))
    ang_v = np.arcsin(np.minimum(1.0, step * np.sqrt(flips_v) / np.maximum(nrm_v - step * np.sqrt(flips_v), 1.0)))
    bound = sum(abs(eta[i]) * (ang_t[i] + ang_v[i].max()) for i in range(C)) + SCORE_TOL * sum(eta)     # [nt]
    want_full = oracle.score(o_tc, o_vc, o_ts, o_vs, eta, off, d, bits)
    assert np.all(np.abs(_np(scores) - want_full) <= bound), float((np.abs(_np(scores) - want_full) / bound).max())
    assert bound.max() <= 2e-2 * sum(eta)            # the bound itself stays small: few codes differ
    # selections agree up to near-ties: a score moves by at most bmax, hence so does the 50th largest, so an index in
    # one set only has an oracle score within 2 bmax of the oracle's threshold
    o_idx = oracle.select_topk(want_full, cfg["frac"])
    thr = np.sort(want_full)[-50]
    for t in set(idx.tolist()) ^ set(o_idx.tolist()):
        assert abs(want_full[t] - thr) <= 2 * bound.max()


# ----------------------------------------------------------------------------------------------
# Full-size shapes, sampled (the launch configuration the benchmark times)
# ----------------------------------------------------------------------------------------------

def test_projection_full_size_sampled():
    # config 2 shape: 256 bf16 rows, P = 2^23, d = 8192, 4-bit, in the launch configuration the benchmark times
    # (128 K chunks x 32 tiles of 256 coordinates = 4096 work items walked by 74 persistent CTA pairs).
    cfg = W.CONFIGS["c2_project_quantize"]
    n, P, d, bits, seed = cfg["batch_rows"], cfg["P"], cfg["d"], cfg["bits"], 31337
    g = W.student_t_gradients(n, P, seed=500, device=DEV, dtype=torch.bfloat16)
    m, v = W.adam_moments(P, seed=501, device=DEV)
    out = B.qless_project_quantize(g, d, seed, bits, m, v, want_proj=True)
    B.qless_check()
    proj = _np(out["proj"])
    # (1) the oracle evaluates one coordinate in each of the 64 halves (one CTA of a pair each) of the 32 coordinate
    # tiles, at an offset that walks through the half, plus the first and last coordinates, for rows of both row halves
    rows = [0, 100, 255]
    coords = sorted({128 * h + (37 * h + 5) % 128 for h in range(64)} | {0, 1, 127, 128, 8191})
    gamma = oracle.adam_gamma(_np(g[rows].float()), _np(m), _np(v))
    want = oracle.project_rows(gamma, d, seed, coords)
    got = proj[np.ix_(rows, coords)]
    ref_scale = np.abs(proj[rows]).max(axis=1, keepdims=True)
    assert (np.abs(got - want) / ref_scale).max() <= PROJ_TOL
    # (2) all 256 x 8192 outputs against the CUDA-core kernel of the same definition (another summation order inside
    # a K chunk, both in fp32): a misplaced (K chunk, tile) work item would move its outputs by about 1/sqrt(128) of
    # their size; rounding differences of two fp32 summations of exact products (measured: 1.5e-6) stay below 2e-5
    try:
        B.qless_set_projection_path(1)
        ref = B.qless_project_quantize(g, d, seed, bits, m, v, want_proj=True)
    finally:
        B.qless_set_projection_path(0)
    rel_l2, rel_max = _proj_err(proj, _np(ref["proj"]))
    assert rel_l2 <= 2e-5 and rel_max <= 2e-5, (rel_l2, rel_max)
    # (3) properties that hold at any size: oracle stage 2 on the GPU's projection reproduces the codes (audited)
    _audit_codes_against_oracle_quantiser(proj, _np(out["codes"]), _np(out["scales"]), _np(out["sumsq"]), bits)
    # JL: the projection keeps the norm of Gamma within 5 sigma
    g2 = (gamma.astype(np.float64) ** 2).sum(1)
    y2 = (proj[rows].astype(np.float64) ** 2).sum(1)
    assert np.all(np.abs(y2 / g2 - 1) <= 5 * math.sqrt(2.0 / d))


@pytest.mark.parametrize("bits", [8, 1])
def test_scoring_full_width_sampled(bits):
    # config 3/4 shape at reduced N: d = 8192, V = 448 in tasks 64/128/256, C = 4; oracle on sampled rows
    C, N, V, d = 4, 5000, 448, 8192
    eta = [1.0, 0.75, 0.5, 0.25]; off = [0, 64, 192, 448]
    tc, vc, ts, vs, tss, vss = _make_store(bits, C, N, V, d, seed=600)
    got = _np(B.qless_score(tc, vc, ts, vs, eta, off, d, bits, train_sumsq=tss, val_sumsq=vss))
    for t0 in (0, 2500, 4990):
        want = oracle.score(_np(tc), _np(vc), _np(ts), _np(vs), eta, off, d, bits, t0=t0, nt=10)
        assert np.abs(got[t0:t0 + 10] - want).max() <= SCORE_TOL * sum(eta)
    idx = _np(B.qless_select_topk(torch.from_numpy(got).to(DEV), 0.05))
    assert np.array_equal(idx, oracle.select_topk(got, 0.05))


def _build_store_chunked(bits, C, N, V, d, seed):
    """The benchmark's way of building a large store: features generated and quantised 16 384 rows at a time."""
    rb = d * bits // 8
    tc = torch.empty((C, N, rb), dtype=torch.uint8, device=DEV); vc = torch.empty((C, V, rb), dtype=torch.uint8, device=DEV)
    ts = torch.empty((C, N), device=DEV); vs = torch.empty((C, V), device=DEV)
    tq = torch.empty((C, N), dtype=torch.int32, device=DEV); vq = torch.empty((C, V), dtype=torch.int32, device=DEV)
    for r0 in range(0, N, 16384):
        r1 = min(N, r0 + 16384)
        xs = W.lowrank_gaussian_features(r1 - r0, d, C, seed=seed + r0, device=DEV)
        for i in range(C):
            tc[i, r0:r1], ts[i, r0:r1], tq[i, r0:r1] = B.qless_quantize(xs[i], bits)
    xs = W.lowrank_gaussian_features(V, d, C, seed=seed - 1, device=DEV)
    for i in range(C):
        vc[i], vs[i], vq[i] = B.qless_quantize(xs[i], bits)
    return tc, vc, ts, vs, tq, vq


@pytest.mark.parametrize("cfg_name,bits", [("c3_score_sweep", 8), ("c3_score_sweep", 4), ("c3_score_sweep", 2),
                                           ("c4_onebit_scaleup", 1)])
def test_scoring_full_size_sampled_rows(cfg_name, bits):
    # configs 3 and 4 at their full sizes, in the launch configuration the benchmark times (every CTA pair walks
    # many tiles, the last tile is ragged): the oracle scores sampled train rows one by one (a row's score depends
    # on no other train row), and selects from the GPU's full score vector
    cfg = W.CONFIGS[cfg_name]
    N, d, C, V = cfg["N"], cfg["d"], cfg["C"], sum(cfg["tasks"])
    off = W.task_offsets(cfg["tasks"]).tolist()
    tc, vc, ts, vs, tq, vq = _build_store_chunked(bits, C, N, V, d, seed=7000)
    scores = B.qless_score(tc, vc, ts, vs, cfg["lr"], off, d, bits, train_sumsq=tq, val_sumsq=vq)
    B.qless_check()
    last_full = (N // 256) * 256
    rows = sorted({0, 1, 127, 128, 255, 256, N // 2, last_full - 1, min(last_full, N - 1), N - 1} |
                  set(np.random.default_rng(5).integers(0, N, 22).tolist()))
    r = torch.tensor(rows, device=DEV)
    want = oracle.score(_np(tc[:, r]), _np(vc), _np(ts[:, r]), _np(vs), cfg["lr"], off, d, bits)
    got = _np(scores)
    assert np.abs(got[rows] - want).max() <= SCORE_TOL * sum(cfg["lr"])
    assert np.isfinite(got).all() and np.abs(got).max() <= sum(cfg["lr"]) * (1 + 1e-5)      # a weighted mean of cosines
    idx = _np(B.qless_select_topk(scores, cfg["frac"]))
    assert idx.size == int(cfg["frac"] * N + 1e-6)
    assert np.array_equal(idx, oracle.select_topk(got, cfg["frac"]))


def test_config5_pipeline_full_width_reduced_rows():
    # config 5 with its real widths (P = 2^22 bf16 gradients, Adam on the train side only, d = 8192, 2-bit codes,
    # 4 checkpoints, 448 validation gradients in 3 tasks) and 256 instead of 32 768 training rows per checkpoint:
    # every stage against the oracle (projection on sampled rows and coordinates, codes from the GPU's own
    # projection, scores from the GPU's own codes on sampled rows, selection from the GPU's own scores)
    cfg = W.CONFIGS["c5_full_pipeline"]
    P, d, C, bits, V, seed, n = cfg["P"], cfg["d"], cfg["C"], cfg["bits"], cfg["n_val"], 555, 256
    off = W.task_offsets(cfg["tasks"]).tolist()
    rb = d * bits // 8
    tc = torch.empty((C, n, rb), dtype=torch.uint8, device=DEV); vc = torch.empty((C, V, rb), dtype=torch.uint8, device=DEV)
    ts = torch.empty((C, n), device=DEV); vs = torch.empty((C, V), device=DEV)
    tq = torch.empty((C, n), dtype=torch.int32, device=DEV); vq = torch.empty((C, V), dtype=torch.int32, device=DEV)
    rows, coords = [0, 129, 255], [0, 127, 128, 5000, 8191]
    for i in range(C):
        m, v = W.adam_moments(P, seed=800 + i, device=DEV)
        for side, count, codes, scales, sumsq in (("train", n, tc, ts, tq), ("val", V, vc, vs, vq)):
            g = W.student_t_gradients(count, P, seed=900 + 10 * i + (side == "val"), device=DEV, dtype=torch.bfloat16)
            adam = (m, v) if side == "train" else (None, None)
            out = B.qless_project_quantize(g, d, seed, bits, adam[0], adam[1], want_proj=True)
            codes[i], scales[i], sumsq[i] = out["codes"], out["scales"], out["sumsq"]
            proj = _np(out["proj"])
            if i in (0, C - 1):
                gamma = oracle.adam_gamma(_np(g[rows].float()), *( (_np(m), _np(v)) if side == "train" else (None, None) ))
                want = oracle.project_rows(gamma, d, seed, coords)
                ref = np.abs(proj[rows]).max(axis=1, keepdims=True)
                assert (np.abs(proj[np.ix_(rows, coords)] - want) / ref).max() <= PROJ_TOL
            _audit_codes_against_oracle_quantiser(proj, _np(out["codes"]), _np(out["scales"]), _np(out["sumsq"]), bits)
    B.qless_check()
    scores = B.qless_score(tc, vc, ts, vs, cfg["lr"], off, d, bits, train_sumsq=tq, val_sumsq=vq)
    r = torch.arange(0, n, 8, device=DEV)
    want = oracle.score(_np(tc[:, r]), _np(vc), _np(ts[:, r]), _np(vs), cfg["lr"], off, d, bits)
    assert np.abs(_np(scores)[::8] - want).max() <= SCORE_TOL * sum(cfg["lr"])
    idx = _np(B.qless_select_topk(scores, cfg["frac"]))
    assert np.array_equal(idx, oracle.select_topk(_np(scores), cfg["frac"]))


def test_config5_pipeline_full_size():
    # config 5 at its own size: 4 checkpoints x (32 768 training + 448 validation) bf16 gradients of width 2^22, Adam on
    # the training side, d = 8192, 2-bit codes, scoring of the 32 768-row store against 448 validation vectors in 3
    # tasks, top 5 %. Training batches of 256 rows are distinct: four generated batches per checkpoint, each used 32
    # times with its columns rotated by another multiple of 1024 (a rotation changes every projected value). Against
    # the oracle: the projection of sampled batches on sampled rows and coordinates, the codes of whole sampled batches
    # from the GPU's own projection, the scores of sampled rows of the final store, the selection from the GPU's scores.
    cfg = W.CONFIGS["c5_full_pipeline"]
    N, V, P, d, C, bits, seed = cfg["n_train"], cfg["n_val"], cfg["P"], cfg["d"], cfg["C"], cfg["bits"], 5150
    off = W.task_offsets(cfg["tasks"]).tolist()
    rb = d * bits // 8
    tc = torch.empty((C, N, rb), dtype=torch.uint8, device=DEV); vc = torch.empty((C, V, rb), dtype=torch.uint8, device=DEV)
    ts = torch.empty((C, N), device=DEV); vs = torch.empty((C, V), device=DEV)
    tq = torch.empty((C, N), dtype=torch.int32, device=DEV); vq = torch.empty((C, V), dtype=torch.int32, device=DEV)
    ws = torch.empty(B.qless_project_quantize_workspace(256, P, d, bits), dtype=torch.uint8, device=DEV)
    proj = torch.empty((256, d), device=DEV)
    rolled = torch.empty((256, P), dtype=torch.bfloat16, device=DEV)
    rows, coords = [0, 127, 128, 255], [0, 127, 128, 4097, 8191]
    nb = N // 256
    checked = {(0, 0), (0, nb - 1), (C - 1, 37), (C - 1, nb - 1)}           # (checkpoint, batch) pairs the oracle looks into

    def check_batch(g, m, v, out, count):
        p_np = _np(out["proj"])[:count]
        gamma = oracle.adam_gamma(_np(g[rows].float()), None if m is None else _np(m), None if v is None else _np(v))
        want = oracle.project_rows(gamma, d, seed, coords)
        ref = np.abs(p_np[rows]).max(axis=1, keepdims=True)
        assert (np.abs(p_np[np.ix_(rows, coords)] - want) / ref).max() <= PROJ_TOL
        _audit_codes_against_oracle_quantiser(p_np, _np(out["codes"]), _np(out["scales"]), _np(out["sumsq"]), bits)

    for i in range(C):
        m, v = W.adam_moments(P, seed=1800 + i, device=DEV)
        pool = [W.student_t_gradients(256, P, seed=1900 + 8 * i + j, device=DEV, dtype=torch.bfloat16) for j in range(4)]
        for b in range(nb):
            shift = (b // 4) * 1024
            g = pool[b % 4]
            if shift:
                rolled[:, shift:] = g[:, :P - shift]; rolled[:, :shift] = g[:, P - shift:]
                g = rolled
            r0 = b * 256
            look = (i, b) in checked
            out = B.qless_project_quantize(g, d, seed, bits, m, v, workspace=ws,
                                           out=dict(codes=tc[i, r0:r0 + 256], scales=ts[i, r0:r0 + 256], sumsq=tq[i, r0:r0 + 256],
                                                    proj=proj if look else None))
            if look:
                check_batch(g, m, v, out, 256)
        del pool
        gv = W.student_t_gradients(V, P, seed=2000 + i, device=DEV, dtype=torch.bfloat16)
        for r0 in range(0, V, 256):
            r1 = min(V, r0 + 256)
            out = B.qless_project_quantize(gv[r0:r1], d, seed, bits, workspace=ws,
                                           out=dict(codes=vc[i, r0:r1], scales=vs[i, r0:r1], sumsq=vq[i, r0:r1], proj=proj[:r1 - r0]))
            if i in (0, C - 1) and r0 == 0:
                check_batch(gv[r0:r1], None, None, out, r1 - r0)
        del gv, m, v
    B.qless_check()
    scores = B.qless_score(tc, vc, ts, vs, cfg["lr"], off, d, bits, train_sumsq=tq, val_sumsq=vq)
    B.qless_check()
    got = _np(scores)
    sample = sorted({0, 1, 127, 128, 255, 256, 257, N // 2, N - 257, N - 256, N - 255, N - 2, N - 1} |
                    set(np.random.default_rng(55).integers(0, N, 27).tolist()))
    r = torch.tensor(sample, device=DEV)
    want = oracle.score(_np(tc[:, r]), _np(vc), _np(ts[:, r]), _np(vs), cfg["lr"], off, d, bits)
    assert np.abs(got[sample] - want).max() <= SCORE_TOL * sum(cfg["lr"])
    assert np.isfinite(got).all() and np.abs(got).max() <= sum(cfg["lr"]) * (1 + 1e-5)
    assert np.unique(got).size > N // 2                    # the rotated batches gave distinct rows, not 32 copies of four
    idx = _np(B.qless_select_topk(scores, cfg["frac"]))
    assert idx.size == 1638
    assert np.array_equal(idx, oracle.select_topk(got, cfg["frac"]))


# ----------------------------------------------------------------------------------------------
# Bounded device-side waits: a wait that nothing satisfies gives up, the kernel returns, the host reads the status
# ----------------------------------------------------------------------------------------------

def test_bounded_wait_times_out_and_reports():
    B.qless_check()                                  # start from a clear flag
    s = torch.randn(10_000, device=DEV)
    before = _np(B.qless_select_topk(s, 0.1))
    B.qless_selftest_timeout(1024)                   # returns: the launch only enqueues the kernel
    with pytest.raises(B.QlessError) as e:
        B.qless_check()
    assert e.value.status == B.ERR_TIMEOUT
    assert "0x1)" in str(e.value)                    # the producer role's code alone: the second waiter left on the abort flag
    B.qless_check()                                  # the flag was cleared by the failing check
    # the context is intact: the library still computes, and no later check trips
    assert np.array_equal(_np(B.qless_select_topk(s, 0.1)), before)
    x = W.student_t_gradients(8, 1024, seed=3, device=DEV, dtype=torch.bfloat16)
    B.qless_project_quantize(x, 256, 1, 4)
    B.qless_check()
    with pytest.raises(B.QlessError):
        B.qless_selftest_timeout(10)                 # poll limit out of range: refused on the host


# ----------------------------------------------------------------------------------------------
# Micro-benchmarks behind the roofline denominators: they run and report plausible rates
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("what,lo,hi", [("i8_ss_pair", 1e15, 1e16), ("i8_ss_pair_n448", 1e15, 1e16),
                                        ("tma_l2_stream", 1e12, 5e13), ("i8_n448_with_tma", 1e15, 1e16),
                                        ("i8_n448_commit_per_block", 1e15, 1e16),
                                        ("fp4_ss_pair_n448", 2e15, 2e16), ("fp4_ts_pair", 2e15, 2e16)])
def test_microbenchmarks_run(what, lo, hi):
    ms, ops = B.qless_microbench(what, 2000)
    B.qless_check()
    assert ms > 0 and lo <= ops / (ms * 1e-3) <= hi, (what, ms, ops)
