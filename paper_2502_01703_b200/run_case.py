"""Run one stage of the hot path at a chosen shape on synthetic inputs (for profiling a small case).

    python -m paper_2502_01703_b200.run_case project  --n 256 --P 1048576 --d 8192 --bits 4 --iters 3   (--matrix gaussian)
    python -m paper_2502_01703_b200.run_case quantize --n 32768 --d 8192 --bits 4
    python -m paper_2502_01703_b200.run_case score    --N 20000 --V 448 --C 4 --d 8192 --bits 8     (16: the bf16 baseline)
    python -m paper_2502_01703_b200.run_case select   --N 67108864 --frac 0.05

Prints the CUDA-event time per iteration of the library call.
"""
import argparse

import torch

from . import binding as B
from . import workloads as W


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("stage", choices=["project", "quantize", "score", "select"])
    ap.add_argument("--n", type=int, default=256)
    ap.add_argument("--N", type=int, default=20000)
    ap.add_argument("--V", type=int, default=448)
    ap.add_argument("--C", type=int, default=4)
    ap.add_argument("--P", type=int, default=1 << 20)
    ap.add_argument("--d", type=int, default=8192)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--frac", type=float, default=0.05)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--no-adam", action="store_true")
    ap.add_argument("--matrix", choices=["rademacher", "gaussian"], default="rademacher", help="random matrix of the projection")
    a = ap.parse_args()
    dev = "cuda"
    if a.stage == "project":
        matrix = B.GAUSSIAN if a.matrix == "gaussian" else B.RADEMACHER
        g = W.student_t_gradients(a.n, a.P, seed=1, device=dev, dtype=torch.bfloat16)
        m, v = (None, None) if a.no_adam else W.adam_moments(a.P, seed=2, device=dev)
        ws = torch.empty(B.qless_project_quantize_workspace(a.n, a.P, a.d, a.bits), dtype=torch.uint8, device=dev)
        fn = lambda: B.qless_project_quantize(g, a.d, 7, a.bits, m, v, workspace=ws, matrix=matrix)
    elif a.stage == "quantize":
        x = torch.randn((a.n, a.d), device=dev)
        fn = lambda: B.qless_quantize(x, a.bits)
    elif a.stage == "score":
        sizes = [64, 128, 256] if a.V == 448 else [a.V]
        off = W.task_offsets(sizes).tolist()
        eta = [1.0, 0.75, 0.5, 0.25, 0.2, 0.1, 0.05, 0.01][:a.C]
        sc = torch.empty(a.N, device=dev)
        if a.bits == 16:
            t16 = torch.empty((a.C, a.N, a.d), dtype=torch.bfloat16, device=dev)
            v16 = torch.empty((a.C, a.V, a.d), dtype=torch.bfloat16, device=dev)
            for i in range(a.C):
                for r0 in range(0, a.N, 8192):
                    r1 = min(a.N, r0 + 8192)
                    t16[i, r0:r1] = W.lowrank_gaussian_features(r1 - r0, a.d, 1, seed=100 + i * 1000 + r0, device=dev)[0].to(torch.bfloat16)
                v16[i] = W.lowrank_gaussian_features(a.V, a.d, 1, seed=5 + i, device=dev)[0].to(torch.bfloat16)
            ws = torch.empty(B.qless_score_16bit_workspace(a.N, a.V, a.C, len(sizes)), dtype=torch.uint8, device=dev)
            tn, vn = B.qless_inv_norms_16bit(t16), B.qless_inv_norms_16bit(v16)
            fn = lambda: B.qless_score_16bit(t16, v16, eta, off, scores=sc, workspace=ws, train_inv_norms=tn, val_inv_norms=vn)
        rb = a.d * min(a.bits, 8) // 8
        tc = torch.empty((a.C, a.N if a.bits != 16 else 1, rb), dtype=torch.uint8, device=dev)
        vc = torch.empty((a.C, a.V, rb), dtype=torch.uint8, device=dev)
        ts = torch.empty((a.C, a.N), device=dev); vs = torch.empty((a.C, a.V), device=dev)
        tss = torch.empty((a.C, a.N), dtype=torch.int32, device=dev); vss = torch.empty((a.C, a.V), dtype=torch.int32, device=dev)
        chunk = 8192
        for i in range(a.C if a.bits != 16 else 0):
            for r0 in range(0, a.N, chunk):
                r1 = min(a.N, r0 + chunk)
                x = W.lowrank_gaussian_features(r1 - r0, a.d, 1, seed=100 + i * 1000 + r0, device=dev)[0]
                tc[i, r0:r1], ts[i, r0:r1], tss[i, r0:r1] = B.qless_quantize(x, a.bits)
            x = W.lowrank_gaussian_features(a.V, a.d, 1, seed=5 + i, device=dev)[0]
            vc[i], vs[i], vss[i] = B.qless_quantize(x, a.bits)
        if a.bits != 16:
            ws = torch.empty(B.qless_score_workspace(a.N, a.V, a.C, len(sizes), a.d, a.bits), dtype=torch.uint8, device=dev)
            fn = lambda: B.qless_score(tc, vc, ts, vs, eta, off, a.d, a.bits, train_sumsq=tss, val_sumsq=vss, scores=sc, workspace=ws)
    else:
        s = torch.randn(a.N, device=dev)
        idx = torch.empty(a.N, dtype=torch.int64, device=dev)
        ws = torch.empty(B.qless_select_topk_workspace(a.N), dtype=torch.uint8, device=dev)
        fn = lambda: B.qless_select_topk(s, a.frac, indices=idx, workspace=ws)
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    B.qless_check()
    print(f"{a.stage}: {e0.elapsed_time(e1) / a.iters:.4f} ms per call")


if __name__ == "__main__":
    main()
