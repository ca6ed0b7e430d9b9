"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random inputs (torch generators, on whichever device it
is asked for). It holds none of the method's arithmetic, which is why both the
CUDA tests/benchmark and the CPU oracle's tests may use it: whatever it returns
is handed to both sides as the same bytes.

Shapes follow the paper: per-example LoRA gradients of dimension P, projected to
d = 8192 features, C = 4 warm-up checkpoints, about 270 K training examples and
a few hundred validation examples grouped in target tasks (Sec. 4.1).
"""
import math

import torch


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def student_t_gradients(n, P, seed, device="cpu", dtype=torch.float32, nu=3, chunk_rows=None):
    """Heavy-tailed per-example gradients: entry = s_row * t, t ~ Student-t(nu) drawn as
    Z / sqrt(chi2_nu / nu), s_row ~ lognormal(0, 1). Returns [n, P] of `dtype`."""
    gen = _gen(seed, device)
    out = torch.empty((n, P), dtype=dtype, device=device)
    if n == 0:
        return out
    row_scale = torch.exp(torch.randn((n, 1), generator=gen, device=device, dtype=torch.float32))
    if chunk_rows is None:
        chunk_rows = max(1, min(n, (1 << 26) // max(P, 1)))
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        z = torch.randn((r1 - r0, P), generator=gen, device=device, dtype=torch.float32)
        chi = torch.zeros_like(z)
        for _ in range(nu):
            w = torch.randn((r1 - r0, P), generator=gen, device=device, dtype=torch.float32)
            chi.addcmul_(w, w)
        t = z / torch.sqrt(chi / nu)
        out[r0:r1] = (t * row_scale[r0:r1]).to(dtype)
    return out


def adam_moments(P, seed, device="cpu"):
    """Optimizer state of one checkpoint: m ~ N(0, sigma=1e-3), v = |N(0, sigma=1e-6)|, fp32 [P]."""
    gen = _gen(seed, device)
    m = torch.randn(P, generator=gen, device=device, dtype=torch.float32) * 1e-3
    v = (torch.randn(P, generator=gen, device=device, dtype=torch.float32) * 1e-6).abs()
    return m, v


def lowrank_gaussian_features(N, d, C, seed, device="cpu", rank=32, rho=0.5, chunk_rows=1 << 15,
                              out=None):
    """Projected-gradient features for a scoring workload, fp32 [C, N, d], unit rows:
    x = sqrt(1-rho) z / sqrt(d) + sqrt(rho) (U c) / sqrt(rank), z ~ N(0, I_d) fresh per
    (example, checkpoint), U in R^{d x rank} ~ N(0, 1/d) fixed per seed, c ~ N(0, I_rank) fixed per
    example across checkpoints; then scaled to unit length."""
    gen = _gen(seed, device)
    U = torch.randn((d, rank), generator=gen, device=device, dtype=torch.float32) / math.sqrt(d)
    if out is None:
        out = torch.empty((C, N, d), dtype=torch.float32, device=device)
    for r0 in range(0, N, chunk_rows):
        r1 = min(N, r0 + chunk_rows)
        c = torch.randn((r1 - r0, rank), generator=gen, device=device, dtype=torch.float32)
        low = (c @ U.t()) * math.sqrt(rho / rank)
        for i in range(C):
            z = torch.randn((r1 - r0, d), generator=gen, device=device, dtype=torch.float32)
            x = z * math.sqrt((1.0 - rho) / d) + low
            out[i, r0:r1] = x / x.norm(dim=1, keepdim=True)
    return out


def task_offsets(sizes):
    """[T+1] int32 prefix offsets of validation tasks with the given sizes."""
    off = [0]
    for s in sizes:
        off.append(off[-1] + int(s))
    return torch.tensor(off, dtype=torch.int32)


# The five named configurations (sizes only; generators above supply the values).
CONFIGS = {
    "c1_tiny_e2e": dict(n_train=1000, n_val=64, P=8192, d=512, C=2, bits=8, lr=[1.0, 0.5],
                        tasks=[32, 32], frac=0.05, grad_dtype="f32"),
    "c2_project_quantize": dict(batches=64, batch_rows=256, P=1 << 23, d=8192, bits=4, grad_dtype="bf16"),
    "c3_score_sweep": dict(N=270_000, d=8192, C=4, bits=[8, 4, 2, 1], tasks=[64, 128, 256],
                           lr=[1.0, 0.75, 0.5, 0.25], frac=0.05),
    "c4_onebit_scaleup": dict(N=2_000_000, d=8192, C=4, bits=1, tasks=[64, 128, 256],
                              lr=[1.0, 0.75, 0.5, 0.25], frac=0.01),
    "c5_full_pipeline": dict(n_train=32_768, n_val=448, P=1 << 22, d=8192, C=4, bits=2,
                             tasks=[64, 128, 256], lr=[1.0, 0.75, 0.5, 0.25], frac=0.05,
                             grad_dtype="bf16"),
}
