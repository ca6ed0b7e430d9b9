#!/usr/bin/env python
"""Benchmark of the QLESS hot path: gradients projected + quantised per second at P = 2^23, d = 8192.

One step = one batch of 256 bf16 per-example gradients through the whole path: Adam prologue ->
Philox-Rademacher projection -> normalise -> 4-bit absmax codes (qless_project_quantize), then the
batch's codes scored against a resident 448-vector validation store in 3 tasks (qless_score) and the
top 5 % selected (qless_select_topk). Inputs are seeded synthetic data (Student-t(3) entries with
lognormal row scales); the batch (4.3 GB) is far larger than L2, so no flush is needed between steps.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0). With --gpus N > 1 (launched by torch.distributed.run, one rank per
GPU) every rank works on its own batches: weak scaling, no data-path collective.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes of one projection launch per projected coordinate (dram__bytes_read.sum + dram__bytes_write.sum of
# project_tc_kernel): one ncu capture at n = 256, d = 8192, P = 2^22 (the smallest P with the K-chunk length of the
# benchmark's P = 2^23) gave 2.9665 GB + 120.6 MB; both parts grow in proportion to P (the Gamma batch read, and one fp32
# partial per 262 144-coordinate chunk written).
PROJECT_TRAFFIC_BYTES_PER_P = (2.966501e9 + 120.602368e6) / 4194304.0
PROJECT_TRAFFIC_SOURCE = "ncu capture at n=256, d=8192, P=2^22, scaled by P (profiles/project_tc_kernel__n256_P2e22_d8192.md)"
WORKLOAD = "c2_project_quantize"
N_VAL, TASKS, FRAC = 448, [64, 128, 256], 0.05
SEED = 20250203


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        return dict(sm_mhz=sm[len(sm) // 2] if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def bench_config(cfg):
    """The `config` object of the JSON line, the same for both arms."""
    return dict(workload=WORKLOAD, batch_rows=cfg["batch_rows"], P=cfg["P"], d=cfg["d"], bits=cfg["bits"], val_rows=N_VAL,
                tasks=TASKS, select_frac=FRAC, l2="inputs larger than L2 (4.3 GB batch), no flush")


def host_cores():
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def _threaded(fn, pieces, threads):
    """Runs fn(piece) for every piece on `threads` host threads. The oracle's C functions are called through ctypes,
    which releases the interpreter lock for the duration of the call, so the pieces run on separate cores; each call
    is the unchanged single-threaded oracle routine on its own rows or coordinates."""
    if threads <= 1:
        return [fn(p) for p in pieces]
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(fn, pieces))


class OracleProjectionSample:
    """The oracle on a bounded sample of the benchmark's workload: n_rows gradient rows at full P through the Adam
    prologue, the projection onto n_coords of the d output coordinates (the oracle regenerates a row of R per
    coordinate, so its work is linear in the coordinates taken) and normalise + quantise of full rows. Both the
    reference arm and the cpu_baseline leg time exactly this, so their figures agree."""

    def __init__(self, threads, n_rows=2, coords_per_thread=8):
        import numpy as np
        import torch
        from paper_2502_01703_b200 import workloads as W
        cfg = W.CONFIGS[WORKLOAD]
        self.P, self.d, self.bits = cfg["P"], cfg["d"], cfg["bits"]
        self.threads, self.n_rows = threads, n_rows
        self.n_coords = min(self.d, coords_per_thread * threads)
        self.g = W.student_t_gradients(n_rows, self.P, seed=SEED, dtype=torch.bfloat16).float().numpy()
        self.m, self.v = [t.numpy() for t in W.adam_moments(self.P, seed=SEED + 1)]
        step = self.d // self.n_coords
        self.coords = np.arange(self.n_coords, dtype=np.int32) * step
        self.np = np

    def run(self):
        """One pass over the sample. Returns (seconds one gradient would take through the full path, seconds taken)."""
        import oracle
        np = self.np
        t0 = time.perf_counter()
        gam = np.concatenate(_threaded(lambda r: oracle.adam_gamma(self.g[r:r + 1], self.m, self.v), range(self.n_rows), self.threads))
        t1 = time.perf_counter()
        pieces = np.array_split(self.coords, min(self.threads, self.n_coords))
        y = np.concatenate(_threaded(lambda c: oracle.project_rows(gam, self.d, SEED, c), pieces, self.threads), axis=1)
        t2 = time.perf_counter()
        full = np.resize(y, (self.n_rows, self.d)).astype(np.float32)
        oracle.quantize_rows(full, self.bits, normalize=True)
        t3 = time.perf_counter()
        per_grad = ((t1 - t0) + (t2 - t1) * (self.d / self.n_coords) + (t3 - t2)) / self.n_rows
        return per_grad, t3 - t0

    def describe(self):
        return (f"{self.n_rows} gradient rows at full P=2^23: Adam prologue, projection onto {self.n_coords} of {self.d} output "
                f"coordinates (scaled x{self.d // self.n_coords}; the work is linear in d), normalise+quantise of full rows; "
                f"{self.threads} thread(s) over coordinates")


def run_reference(args):
    """The CPU oracle timed as it stands on a bounded sample of the same workload (rank 0 only; other ranks leave)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2502_01703_b200 import workloads as W
    cfg = W.CONFIGS[WORKLOAD]
    cores = host_cores()
    smp = OracleProjectionSample(cores)
    for _ in range(args.warmup):
        smp.run()
    runs = [smp.run() for _ in range(args.steps)]
    sec = sum(r[0] for r in runs) / len(runs)               # seconds per gradient through the full path
    step_s = sum(r[1] for r in runs) / len(runs)            # seconds a step (one pass over the sample) really took
    value = 1.0 / sec
    line = dict(impl="reference", metric="grads projected+quantized/s (P=2^23,d=8192)", value=value, unit="grads/s",
                n_gpus=args.gpus, steps=args.steps, warmup=args.warmup, ms_per_step=step_s * 1e3,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=bench_config(cfg),
                gradients_per_step=step_s / sec,
                cpu_baseline=dict(value=value, unit="grads/s", cores=cores, kind="oracle", sample=smp.describe()),
                e2e=dict(value=value, unit="grads/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def cpu_baseline():
    """The oracle, as it stands, on the host cores: the projection + quantisation sample of the reference arm (all
    cores and one thread), scoring per code width on sampled train rows of configs 3 and 4 against all 448 x 4
    validation vectors (one thread and all cores, rows split over threads), and selection at the full sizes."""
    import numpy as np
    import oracle
    from paper_2502_01703_b200 import workloads as W
    cores = host_cores()
    t_begin = time.perf_counter()
    smp = OracleProjectionSample(cores)
    smp.run()
    per_grad = min(smp.run()[0] for _ in range(2))
    one = OracleProjectionSample(1, coords_per_thread=16)
    per_grad_1 = one.run()[0]
    out = dict(value=1.0 / per_grad, unit="grads/s", cores=cores, kind="oracle", sample=smp.describe(),
               one_thread=dict(value=1.0 / per_grad_1, unit="grads/s", cores=1, sample=one.describe()))
    # scoring: sampled train rows x all validation vectors x all checkpoints
    cfg = W.CONFIGS["c3_score_sweep"]
    d, C, V = cfg["d"], cfg["C"], sum(cfg["tasks"])
    off = W.task_offsets(cfg["tasks"]).tolist()
    n1, nall = 128, max(256, 16 * cores)
    xt = W.lowrank_gaussian_features(nall, d, C, seed=SEED + 7).numpy()
    xv = W.lowrank_gaussian_features(V, d, C, seed=SEED + 8).numpy()
    scoring = {}
    for b in cfg["bits"]:
        tq = [oracle.quantize_rows(xt[i], b) for i in range(C)]
        vq = [oracle.quantize_rows(xv[i], b) for i in range(C)]
        tc, ts = np.stack([q[0] for q in tq]), np.stack([q[1] for q in tq])
        vc, vs = np.stack([q[0] for q in vq]), np.stack([q[1] for q in vq])

        def part(r, tc=tc, ts=ts, vc=vc, vs=vs, b=b):
            return oracle.score(np.ascontiguousarray(tc[:, r[0]:r[1]]), vc, np.ascontiguousarray(ts[:, r[0]:r[1]]), vs, cfg["lr"], off, d, b)
        t0 = time.perf_counter()
        part((0, n1))
        t1 = time.perf_counter()
        edges = np.linspace(0, nall, cores + 1).astype(int)
        _threaded(part, [(int(edges[k]), int(edges[k + 1])) for k in range(cores) if edges[k + 1] > edges[k]], cores)
        t2 = time.perf_counter()
        scoring[str(b)] = dict(scores_per_s_one_thread=n1 * V / (t1 - t0), scores_per_s_all_cores=nall * V / (t2 - t1),
                               rows_one_thread=n1, rows_all_cores=nall)
    out["scoring_c3_c4"] = dict(per_bits=scoring, cores=cores,
                                sample=(f"{n1} (one thread) / {nall} (all cores) sampled train rows x {V} validation vectors x {C} "
                                        f"checkpoints at d={d}; a score = one (train, validation) pair aggregated over the checkpoints; "
                                        f"the oracle's time per train row does not depend on N, so config 4 (1-bit) has the 1-bit rate"))
    sel = {}
    for name, N, frac in (("c3_270000_top5pct", 270_000, 0.05), ("c4_2000000_top1pct", 2_000_000, 0.01)):
        sc = np.random.default_rng(SEED).standard_normal(N).astype(np.float32)
        t0 = time.perf_counter()
        oracle.select_topk(sc, frac)
        sel[name] = dict(ms=(time.perf_counter() - t0) * 1e3, cores=1)
    out["select"] = dict(sizes=sel, note="full size; the oracle's selection is one sort, so one thread is all it uses")
    out["seconds_spent"] = time.perf_counter() - t_begin
    return out


def max_over_ranks(ms_local, dist=None, device=None):
    """Timing rule for N > 1: every rank measures its own replica on its own device; the job's time is the
    slowest rank's (all-reduce MAX). Replicas share no data, so this is the only collective of the benchmark."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms_local)
    import torch
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step, steps, world, ms_total):
    """Weak scaling: every rank processes its own units; value = all ranks' units / slowest rank's time."""
    return world * units_per_rank_per_step * steps / (ms_total * 1e-3)


def _time_ms(torch, fn, iters, warm=1):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def pipeline_c5(torch, B, W, dev):
    """Config 5 end to end: per checkpoint 32 768 training gradients (P = 2^22, bf16, Adam prologue) and 448
    validation gradients are projected to d = 8192 and stored as 2-bit codes, then scored and the top 5 % selected.
    The gradients are streamed in batches of 256 rows; to keep input generation out of the way each checkpoint
    cycles a pool of 4 generated batches (32 distinct pools over the run), so rows repeat inside a checkpoint: this
    changes nothing in the work done. Times are the library's own per-kernel CUDA-event totals."""
    cfg = W.CONFIGS["c5_full_pipeline"]
    N, V, P, d, C, bits = cfg["n_train"], cfg["n_val"], cfg["P"], cfg["d"], cfg["C"], cfg["bits"]
    rb = d * bits // 8
    off = W.task_offsets(cfg["tasks"]).tolist()
    tc = torch.empty((C, N, rb), dtype=torch.uint8, device=dev); ts = torch.empty((C, N), device=dev)
    tq = torch.empty((C, N), dtype=torch.int32, device=dev)
    vc = torch.empty((C, V, rb), dtype=torch.uint8, device=dev); vs = torch.empty((C, V), device=dev)
    vq = torch.empty((C, V), dtype=torch.int32, device=dev)
    ws = torch.empty(B.qless_project_quantize_workspace(V, P, d, bits), dtype=torch.uint8, device=dev)
    B.qless_profile_collect()
    B.qless_profile_enable(True)
    for i in range(C):
        m, v = W.adam_moments(P, seed=SEED + 300 + i, device=dev)
        pool = [W.student_t_gradients(256, P, seed=SEED + 400 + 8 * i + j, device=dev, dtype=torch.bfloat16) for j in range(4)]
        for b in range(N // 256):
            r0 = b * 256
            B.qless_project_quantize(pool[b % 4], d, SEED, bits, m, v, workspace=ws,
                                     out=dict(codes=tc[i, r0:r0 + 256], scales=ts[i, r0:r0 + 256], sumsq=tq[i, r0:r0 + 256]))
        del pool
        g = W.student_t_gradients(V, P, seed=SEED + 500 + i, device=dev, dtype=torch.bfloat16)
        B.qless_project_quantize(g, d, SEED, bits, workspace=ws, out=dict(codes=vc[i], scales=vs[i], sumsq=vq[i]))
        del g, m, v
    sc = torch.empty(N, device=dev)
    wsc = torch.empty(B.qless_score_workspace(N, V, C, len(off) - 1, d, bits), dtype=torch.uint8, device=dev)
    B.qless_score(tc, vc, ts, vs, cfg["lr"], off, d, bits, train_sumsq=tq, val_sumsq=vq, scores=sc, workspace=wsc)
    idx = B.qless_select_topk(sc, cfg["frac"])
    torch.cuda.synchronize()
    prof = B.qless_profile_collect()
    B.qless_profile_enable(False)
    B.qless_check()
    stages = {k: dict(ms=ms, calls=c) for k, (ms, c) in prof.items()}
    total = sum(ms for ms, _ in prof.values())
    rows = C * (N + V)
    return dict(stages=stages, total_ms=total, gradients=rows, gradients_per_s=rows / (total * 1e-3), selected=int(idx.numel()),
                project_tflops=2.0 * rows * P * d / (prof["project"][0] * 1e-3) / 1e12 if "project" in prof else None,
                note="library time only (per-kernel CUDA events); input generation excluded")


def stage_measurements(torch, B, W, dev, peaks):
    """The other kernels of the path at the sizes where their roofline is observable: quantise on 65 536 rows,
    scoring on the 270 K x 448 x 4-checkpoint store per bit width and on the 2 M-row 1-bit store, selection on
    2^28 scores. Each entry gives the CUDA-event time of the library call and the achieved fraction of the
    relevant measured peak (HBM copy bandwidth, or the library's own tcgen05 int8 / XOR+POPC micro-benchmark)."""
    out = {}
    # measured peaks of the units that have no externally measured figure (int8 tensor pipe, integer ALU mix)
    ms, ops = B.qless_microbench("i8_ss_pair", 20000, device=dev)
    i8_peak = ops / ms / 1e9            # Tops/s
    ms, ops = B.qless_microbench("popc", 20000, device=dev)
    popc_peak = ops / ms / 1e9          # T word-ops/s
    ms, ops = B.qless_microbench("bf16_ts_pair", 20000, device=dev)
    bf16_peak = ops / ms / 1e9          # TFLOP/s
    ms, ops = B.qless_microbench("i8_ss_pair_n448", 20000, device=dev)
    i8_n448 = ops / ms / 1e9            # Tops/s in the two-MMA shape of 8-bit scoring at 448 validation vectors
    # e2m1 operands (kind::mxf4, unit scale factors), the path of 2- and 1-bit scoring: the two-MMA shape with both operands
    # in shared memory (what the kernel issues), and with A in tensor memory (for which a 448-column accumulator leaves no room)
    ms, ops = B.qless_microbench("fp4_ss_pair_n448", 20000, device=dev)
    fp4_n448 = ops / ms / 1e9
    ms, ops = B.qless_microbench("fp4_ts_pair", 20000, device=dev)
    fp4_ts = ops / ms / 1e9
    ms, byts = B.qless_microbench("tma_l2_stream", 20000, device=dev)
    l2_gbs = byts / ms / 1e6            # GB/s from L2 into shared memory, TMA alone
    out["microbench"] = dict(int8_tops=i8_peak, popc_xor_add_twordops=popc_peak, bf16_tcgen05_tflops=bf16_peak,
                             int8_tops_scoring_shape_n448=i8_n448, fp4_tops_scoring_shape_n448=fp4_n448,
                             fp4_tops_a_in_tensor_memory=fp4_ts, tma_l2_to_smem_gbs=l2_gbs,
                             note="back-to-back tcgen05.mma / XOR+POPC+IADD on all SMs, burst; TMA streaming from an L2-resident buffer")
    # the same int8 micro-benchmark held for about two seconds, clocks sampled: the tensor pipe under the power cap
    smp = ClockSampler(torch.cuda.current_device())
    smp.start()
    ms, ops = B.qless_microbench("i8_ss_pair", 4_000_000, device=dev)
    ck = smp.stop()
    i8_sustained = ops / ms / 1e9
    out["microbench"].update(int8_tops_sustained=i8_sustained, int8_sustained_clocks=ck)
    smp = ClockSampler(torch.cuda.current_device())
    smp.start()
    ms, ops = B.qless_microbench("fp4_ss_pair_n448", 2_000_000, device=dev)
    ck4 = smp.stop()
    fp4_sustained = ops / ms / 1e9
    out["microbench"].update(fp4_tops_scoring_shape_sustained=fp4_sustained, fp4_sustained_clocks=ck4)
    # the int8 MMAs of 8-bit scoring reading, for every K block, operands that TMA has just streamed from a buffer of
    # pseudo-random int8 values: the tensor pipe on data that changes, held for about two seconds with the clocks
    # sampled. This is the sustained figure a scoring kernel can be held against: same shape, same data statistics,
    # no epilogue, no HBM.
    gen = torch.Generator(device=dev); gen.manual_seed(SEED + 11)
    rnd = torch.randint(-127, 128, (4 << 20,), generator=gen, device=dev, dtype=torch.int8).view(torch.uint8)
    B.qless_microbench("i8_n448_streamed_operands", 20000, device=dev, scratch=rnd)
    smp = ClockSampler(torch.cuda.current_device())
    smp.start()
    ms, ops = B.qless_microbench("i8_n448_streamed_operands", 3_000_000, device=dev, scratch=rnd)
    ck_rand = smp.stop()
    i8_random = ops / ms / 1e9
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    out["microbench"].update(int8_tops_random_operands_sustained=i8_random, int8_random_operands_clocks=ck_rand,
                             int8_random_operands_seconds=ms * 1e-3)
    del rnd
    d = 8192
    # ---- quantise ----
    n = 65536
    x = torch.randn((n, d), device=dev)
    q = {}
    for bits in (8, 4, 2, 1):
        t = _time_ms(torch, lambda: B.qless_quantize(x, bits), 5)
        byts = n * (4 * d + d * bits // 8 + 8)
        q[str(bits)] = dict(ms=t, gbs=byts / t / 1e6, frac_of_hbm=byts / t / 1e6 / peaks["hbm_gbs"])
    out["quantize_65536x8192"] = q
    del x
    # ---- scoring, config 3 ----
    cfg = W.CONFIGS["c3_score_sweep"]
    N, C, V = cfg["N"], cfg["C"], sum(cfg["tasks"])
    off = W.task_offsets(cfg["tasks"]).tolist()
    store = {b: dict(tc=torch.empty((C, N, d * b // 8), dtype=torch.uint8, device=dev),
                     vc=torch.empty((C, V, d * b // 8), dtype=torch.uint8, device=dev),
                     ts=torch.empty((C, N), device=dev), vs=torch.empty((C, V), device=dev),
                     tq=torch.empty((C, N), dtype=torch.int32, device=dev), vq=torch.empty((C, V), dtype=torch.int32, device=dev))
             for b in cfg["bits"]}
    t16 = torch.empty((C, N, d), dtype=torch.bfloat16, device=dev)       # the 16-bit store of the same features
    v16 = torch.empty((C, V, d), dtype=torch.bfloat16, device=dev)
    chunk = 16384
    for r0 in range(0, N, chunk):
        r1 = min(N, r0 + chunk)
        xs = W.lowrank_gaussian_features(r1 - r0, d, C, seed=SEED + 7 + r0, device=dev)
        for i in range(C):
            t16[i, r0:r1] = xs[i].to(torch.bfloat16)
            for b in cfg["bits"]:
                st = store[b]
                st["tc"][i, r0:r1], st["ts"][i, r0:r1], st["tq"][i, r0:r1] = B.qless_quantize(xs[i], b)
    xs = W.lowrank_gaussian_features(V, d, C, seed=SEED + 8, device=dev)
    for i in range(C):
        v16[i] = xs[i].to(torch.bfloat16)
        for b in cfg["bits"]:
            st = store[b]
            st["vc"][i], st["vs"][i], st["vq"][i] = B.qless_quantize(xs[i], b)
    del xs
    sc = torch.empty(N, device=dev)
    res = {}
    tops = {}
    for b in cfg["bits"]:
        st = store[b]
        ws = torch.empty(B.qless_score_workspace(N, V, C, len(off) - 1, d, b), dtype=torch.uint8, device=dev)
        t = _time_ms(torch, lambda: B.qless_score(st["tc"], st["vc"], st["ts"], st["vs"], cfg["lr"], off, d, b,
                                                  train_sumsq=st["tq"], val_sumsq=st["vq"], scores=sc, workspace=ws), 5)
        e = dict(ms=t, scores_per_s=N * V / (t * 1e-3), pair_dots_per_s=N * V * C / (t * 1e-3))
        iops = 2.0 * N * V * C * d
        e.update(bound="tensor", achieved_tops=iops / t / 1e9, frac_of_int8_peak=iops / t / 1e9 / i8_peak,
                 tensor_path="e2m1 (kind::mxf4, unit scales)" if b <= 2 else "int8 (kind::i8)",
                 store_gb=C * (N + V) * (d * b // 8 + 8) / 1e9)
        if b <= 2:
            e.update(frac_of_fp4_peak=iops / t / 1e9 / fp4_n448)
        # the same call repeated for over a second with the clocks sampled, against the sustained micro-benchmark
        smp = ClockSampler(torch.cuda.current_device())
        smp.start()
        ts_ = _time_ms(torch, lambda: B.qless_score(st["tc"], st["vc"], st["ts"], st["vs"], cfg["lr"], off, d, b,
                                                    train_sumsq=st["tq"], val_sumsq=st["vq"], scores=sc, workspace=ws), 400, warm=0)
        ck = smp.stop()
        if b == 1:
            sc_1bit = sc.clone()        # for the selected-percentage sweep below
        e.update(ms_sustained=ts_, frac_of_int8_sustained=iops / ts_ / 1e9 / i8_sustained, sustained_clocks=ck,
                 frac_of_int8_random_operands_sustained=iops / ts_ / 1e9 / i8_random)
        if b <= 2:
            e.update(frac_of_fp4_sustained=iops / ts_ / 1e9 / fp4_sustained)
        if ck.get("sm_mhz"):
            # against what the hardware's unit count allows at the SM clock this very loop was granted
            hw_ops = HW_FP4_OP_PER_CLK_SM if b <= 2 else HW_INT8_OP_PER_CLK_SM
            e.update({"frac_of_hw_fp4_at_sampled_clock" if b <= 2 else "frac_of_hw_int8_at_sampled_clock":
                      iops / ts_ / 1e9 / (sms * hw_ops * ck["sm_mhz"] * 1e6 / 1e12)})
        if ck.get("sm_mhz") and ck.get("sm_max_mhz"):
            # the micro-benchmark holds the maximum clock (its operands never change, so it draws little power); the
            # scoring kernel runs under the power cap: its rate against the tensor peak at the clock it actually had
            e.update(frac_of_int8_peak_at_sustained_clock=iops / ts_ / 1e9 / (i8_sustained * ck["sm_mhz"] / ck["sm_max_mhz"]))
        tops[b] = B.qless_select_topk(sc, cfg["frac"])
        res[str(b)] = e
        if b == 1:
            # the XOR + population-count kernel (CUDA cores) on the same store, against the integer-ALU peak
            B.qless_set_score_path(1)
            try:
                t = _time_ms(torch, lambda: B.qless_score(st["tc"], st["vc"], st["ts"], st["vs"], cfg["lr"], off, d, b,
                                                          train_sumsq=st["tq"], val_sumsq=st["vq"], scores=sc, workspace=ws), 3)
            finally:
                B.qless_set_score_path(0)
            wops = N * V * C * (d / 32)
            res["1_popc"] = dict(ms=t, scores_per_s=N * V / (t * 1e-3), pair_dots_per_s=N * V * C / (t * 1e-3), bound="alu",
                                 achieved_twordops=wops / t / 1e9, frac_of_popc_peak=wops / t / 1e9 / popc_peak)
    # 16-bit baseline on the same features (timed after the quantised stores, which are the subject): its time, and
    # its top-5 % set as the reference for the overlaps
    sc16 = torch.empty(N, device=dev)
    ws16 = torch.empty(B.qless_score_16bit_workspace(N, V, C, len(off) - 1), dtype=torch.uint8, device=dev)
    tn16, vn16 = B.qless_inv_norms_16bit(t16), B.qless_inv_norms_16bit(v16)      # kept beside the store, like the code norms
    t = _time_ms(torch, lambda: B.qless_score_16bit(t16, v16, cfg["lr"], off, scores=sc16, workspace=ws16,
                                                    train_inv_norms=tn16, val_inv_norms=vn16), 5)
    flops = 2.0 * N * V * C * d
    res["16"] = dict(ms=t, scores_per_s=N * V / (t * 1e-3), pair_dots_per_s=N * V * C / (t * 1e-3), bound="tensor",
                     achieved_tflops=flops / t / 1e9, frac_of_bf16_peak=flops / t / 1e9 / bf16_peak,
                     store_gb=C * (N + V) * d * 2 / 1e9)
    top16 = B.qless_select_topk(sc16, cfg["frac"])
    in16 = torch.zeros(N, dtype=torch.bool, device=dev)
    in16[top16] = True
    del t16, v16, ws16
    # the selected-percentage sweep of the paper's Fig. 4 (0.1 to 10 % with the 1-bit store), on this synthetic store:
    # how much of the 16-bit baseline's selection the 1-bit codes reproduce at each percentage, and the selection time
    sweep = {}
    for frac in (0.001, 0.005, 0.01, 0.02, 0.05, 0.10):
        ref = torch.zeros(N, dtype=torch.bool, device=dev)
        ref[B.qless_select_topk(sc16, frac)] = True
        t = _time_ms(torch, lambda: B.qless_select_topk(sc_1bit, frac), 20)
        sweep[str(frac)] = dict(k=int(frac * N + 1e-6), select_ms=t,
                                overlap_with_16bit=float(ref[B.qless_select_topk(sc_1bit, frac)].float().mean()))
    res["1bit_selected_percentage_sweep"] = sweep
    del sc_1bit
    for b in cfg["bits"]:
        res[str(b)]["top5pct_overlap_with_16bit"] = float(in16[tops[b]].float().mean())
    out["score_c3_270000x448x4"] = res
    # absmean codes of the same features (Sec. 6, Table 3): only the selection overlap is of interest, the kernels
    # that score them are the ones timed above
    del store
    am = {}
    for b in (8, 4, 2):
        tcb = torch.empty((C, N, d * b // 8), dtype=torch.uint8, device=dev); tsb = torch.empty((C, N), device=dev)
        tqb = torch.empty((C, N), dtype=torch.int32, device=dev)
        vcb = torch.empty((C, V, d * b // 8), dtype=torch.uint8, device=dev); vsb = torch.empty((C, V), device=dev)
        vqb = torch.empty((C, V), dtype=torch.int32, device=dev)
        for r0 in range(0, N, chunk):
            r1 = min(N, r0 + chunk)
            xs = W.lowrank_gaussian_features(r1 - r0, d, C, seed=SEED + 7 + r0, device=dev)
            for i in range(C):
                tcb[i, r0:r1], tsb[i, r0:r1], tqb[i, r0:r1] = B.qless_quantize_absmean(xs[i], b)
        xs = W.lowrank_gaussian_features(V, d, C, seed=SEED + 8, device=dev)
        for i in range(C):
            vcb[i], vsb[i], vqb[i] = B.qless_quantize_absmean(xs[i], b)
        del xs
        ws = torch.empty(B.qless_score_workspace(N, V, C, len(off) - 1, d, b), dtype=torch.uint8, device=dev)
        B.qless_score(tcb, vcb, tsb, vsb, cfg["lr"], off, d, b, train_sumsq=tqb, val_sumsq=vqb, scores=sc, workspace=ws)
        topb = B.qless_select_topk(sc, cfg["frac"])
        am[str(b)] = dict(top5pct_overlap_with_16bit=float(in16[topb].float().mean()))
        del tcb, vcb, ws
    out["absmean_c3_overlap"] = am
    idx = torch.empty(N, dtype=torch.int64, device=dev)
    wsel = torch.empty(B.qless_select_topk_workspace(N), dtype=torch.uint8, device=dev)
    out["select_c3_270000_top5pct"] = dict(ms=_time_ms(torch, lambda: B.qless_select_topk(sc, cfg["frac"], indices=idx, workspace=wsel), 20))
    del sc
    # ---- 1-bit scale-up, config 4 ----
    cfg = W.CONFIGS["c4_onebit_scaleup"]
    N = cfg["N"]
    tc = torch.empty((C, N, d // 8), dtype=torch.uint8, device=dev)
    ts = torch.empty((C, N), device=dev); tq = torch.empty((C, N), dtype=torch.int32, device=dev)
    vc = torch.empty((C, V, d // 8), dtype=torch.uint8, device=dev)
    vs = torch.empty((C, V), device=dev); vq = torch.empty((C, V), dtype=torch.int32, device=dev)
    chunk = 32768
    for r0 in range(0, N, chunk):
        r1 = min(N, r0 + chunk)
        xs = W.lowrank_gaussian_features(r1 - r0, d, C, seed=SEED + 9 + r0, device=dev)
        for i in range(C):
            tc[i, r0:r1], ts[i, r0:r1], tq[i, r0:r1] = B.qless_quantize(xs[i], 1)
    xs = W.lowrank_gaussian_features(V, d, C, seed=SEED + 10, device=dev)
    for i in range(C):
        vc[i], vs[i], vq[i] = B.qless_quantize(xs[i], 1)
    del xs
    sc = torch.empty(N, device=dev)
    ws = torch.empty(B.qless_score_workspace(N, V, C, len(off) - 1, d, 1), dtype=torch.uint8, device=dev)
    t = _time_ms(torch, lambda: B.qless_score(tc, vc, ts, vs, cfg["lr"], off, d, 1, train_sumsq=tq, val_sumsq=vq,
                                              scores=sc, workspace=ws), 2)
    iops = 2.0 * N * V * C * d
    out["score_c4_2000000x448x4_1bit"] = dict(ms=t, scores_per_s=N * V / (t * 1e-3), bound="tensor",
                                              achieved_tops=iops / t / 1e9, frac_of_int8_peak=iops / t / 1e9 / i8_peak,
                                              frac_of_fp4_peak=iops / t / 1e9 / fp4_n448, frac_of_fp4_sustained=iops / t / 1e9 / fp4_sustained,
                                              tensor_path="e2m1 (kind::mxf4, unit scales)",
                                              frac_of_int8_random_operands_sustained=iops / t / 1e9 / i8_random)
    # the same store through the XOR + population-count kernel (CUDA cores), against the integer-ALU peak
    B.qless_set_score_path(1)
    try:
        t = _time_ms(torch, lambda: B.qless_score(tc, vc, ts, vs, cfg["lr"], off, d, 1, train_sumsq=tq, val_sumsq=vq,
                                                  scores=sc, workspace=ws), 2)
    finally:
        B.qless_set_score_path(0)
    wops = N * V * C * (d / 32)
    out["score_c4_2000000x448x4_1bit_popc"] = dict(ms=t, scores_per_s=N * V / (t * 1e-3), bound="alu",
                                                   achieved_twordops=wops / t / 1e9, frac_of_popc_peak=wops / t / 1e9 / popc_peak)
    idx = torch.empty(N, dtype=torch.int64, device=dev)
    wsel = torch.empty(B.qless_select_topk_workspace(N), dtype=torch.uint8, device=dev)
    out["select_c4_2000000_top1pct"] = dict(ms=_time_ms(torch, lambda: B.qless_select_topk(sc, cfg["frac"], indices=idx, workspace=wsel), 20))
    del tc, sc, idx
    # ---- config 5: the whole path for a 4-checkpoint store, stage by stage ----
    out["pipeline_c5"] = pipeline_c5(torch, B, W, dev)
    # ---- selection at a size where HBM bandwidth is observable ----
    N = 1 << 28
    s = torch.randn(N, device=dev)
    idx = torch.empty(N // 16, dtype=torch.int64, device=dev)
    wsel = torch.empty(B.qless_select_topk_workspace(N), dtype=torch.uint8, device=dev)
    t = _time_ms(torch, lambda: B.qless_select_topk(s, 0.05, indices=idx, workspace=wsel), 20, warm=2)
    out["select_2^28_top5pct"] = dict(ms=t, gbs_algorithmic=4.0 * N / t / 1e6, frac_of_hbm=4.0 * N / t / 1e6 / peaks["hbm_gbs"],
                                      note="algorithmic bytes = 4N (every score read once)")
    del s, idx, wsel
    # ---- projection with the Gaussian matrix (the distribution Sec. 2.4 names beside Rademacher) ----
    n, P = 256, 1 << 20
    g = W.student_t_gradients(n, P, seed=SEED + 600, device=dev, dtype=torch.bfloat16)
    ws = torch.empty(B.qless_project_quantize_workspace(n, P, d, 4), dtype=torch.uint8, device=dev)
    pq = {}
    for name, kind in (("rademacher", B.RADEMACHER), ("gaussian", B.GAUSSIAN)):
        try:
            B.qless_profile_collect()
            B.qless_profile_enable(True)
            for _ in range(4):
                B.qless_project_quantize(g, d, SEED, 4, workspace=ws, matrix=kind)
            torch.cuda.synchronize()
            prof = B.qless_profile_collect()
        finally:
            B.qless_profile_enable(False)
        t = prof["project"][0] / prof["project"][1]
        pq[name] = dict(ms=t, tflops=2.0 * n * P * d / t / 1e9, grads_per_s=n / (t * 1e-3))
    pq["note"] = "projection kernel alone, 256 bf16 rows, P = 2^20; the Gaussian matrix is bounded by its generator warps"
    out["project_256x2^20_by_matrix"] = pq
    B.qless_check()
    return out


# Tensor-pipe rates the hardware cannot exceed: dense bf16 (fp32 accumulation) 8192 flop and int8 16384 operations per
# clock per SM (the unit counts behind the nominal 2.25 / 4.5 Pop/s at the nominal clock); times the SM count and a clock.
HW_BF16_FLOP_PER_CLK_SM = 8192.0
HW_INT8_OP_PER_CLK_SM = 16384.0
HW_FP4_OP_PER_CLK_SM = 32768.0         # block-scaled e2m1: twice the int8 count (nominal 9 Pop/s dense)


def roofline_entry(achieved_tflops, peaks, clocks, sm_count=148):
    """Roofline object of the projection kernel. `frac` is against the measured sustained library GEMM (the kernel is
    timed inside a long step); a kernel can beat a library figure, so two denominators that it cannot beat stand
    beside it: the hardware's unit count at the SM clock sampled while the timed region ran, and at the maximum clock."""
    r = dict(bound="tensor", kernel="project", achieved=achieved_tflops, peak=peaks["bf16_sustained"], unit="TFLOP/s",
             frac=(achieved_tflops / peaks["bf16_sustained"]) if achieved_tflops else None,
             peak_source=f"{peaks['source']} (sustained bf16 GEMM of a library; burst {peaks['bf16_burst']})")
    if achieved_tflops:
        r["frac_of_burst_matmul"] = achieved_tflops / peaks["bf16_burst"]
        mx = clocks.get("sm_max_mhz") or 1965.0
        r["hw_peak_at_max_clock"] = sm_count * HW_BF16_FLOP_PER_CLK_SM * mx * 1e6 / 1e12
        r["frac_of_hw_peak_at_max_clock"] = achieved_tflops / r["hw_peak_at_max_clock"]
        if clocks.get("sm_mhz"):
            r["hw_peak_at_sampled_clock"] = sm_count * HW_BF16_FLOP_PER_CLK_SM * clocks["sm_mhz"] * 1e6 / 1e12
            r["frac_of_hw_peak_at_sampled_clock"] = achieved_tflops / r["hw_peak_at_sampled_clock"]
    return r


def summarize(stages, cpu, peaks, step_kernels_ms):
    """Compact per-kernel figures taken from the stage measurements (and the oracle's rates beside them)."""
    def pick(e, keys):
        return {k: e[k] for k in keys if k in e}
    c3 = stages.get("score_c3_270000x448x4", {})
    scoring = {"c3": {}, "c4": {}}
    keys = ("ms", "scores_per_s", "tensor_path", "frac_of_int8_peak", "frac_of_int8_sustained", "frac_of_int8_random_operands_sustained",
            "frac_of_hw_int8_at_sampled_clock", "frac_of_fp4_peak", "frac_of_fp4_sustained", "frac_of_hw_fp4_at_sampled_clock",
            "frac_of_popc_peak", "frac_of_bf16_peak")
    for b in ("8", "4", "2", "1", "1_popc", "16"):
        if b in c3:
            scoring["c3"][b] = pick(c3[b], keys)
    if "score_c4_2000000x448x4_1bit" in stages:
        scoring["c4"]["1"] = pick(stages["score_c4_2000000x448x4_1bit"], keys)
    if "score_c4_2000000x448x4_1bit_popc" in stages:
        scoring["c4"]["1_popc"] = pick(stages["score_c4_2000000x448x4_1bit_popc"], keys)
    mb = stages.get("microbench", {})
    out = dict(scoring=scoring,
               peaks=dict(int8_tops_burst=mb.get("int8_tops"), int8_tops_sustained=mb.get("int8_tops_sustained"),
                          int8_tops_random_operands_sustained=mb.get("int8_tops_random_operands_sustained"),
                          fp4_tops_scoring_shape=mb.get("fp4_tops_scoring_shape_n448"), fp4_tops_scoring_shape_sustained=mb.get("fp4_tops_scoring_shape_sustained"),
                          fp4_tops_a_in_tensor_memory=mb.get("fp4_tops_a_in_tensor_memory"),
                          popc_twordops=mb.get("popc_xor_add_twordops"), bf16_tcgen05_tflops=mb.get("bf16_tcgen05_tflops"),
                          hbm_gbs=peaks["hbm_gbs"], source="library micro-benchmarks (tcgen05 int8, XOR+POPC+IADD); HBM: " + peaks["source"]),
               quantize_65536x8192={b: pick(e, ("ms", "frac_of_hbm")) for b, e in stages.get("quantize_65536x8192", {}).items()},
               step_kernels_ms=step_kernels_ms,
               select={k: pick(stages[k], ("ms", "frac_of_hbm")) for k in ("select_c3_270000_top5pct", "select_c4_2000000_top1pct", "select_2^28_top5pct") if k in stages})
    if cpu and "scoring_c3_c4" in cpu:
        out["scoring_cpu_oracle_scores_per_s"] = {b: pick(e, ("scores_per_s_one_thread", "scores_per_s_all_cores"))
                                                  for b, e in cpu["scoring_c3_c4"]["per_bits"].items()}
        out["scoring_cpu_oracle_cores"] = cpu["scoring_c3_c4"]["cores"]
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2502_01703_b200 import binding as B
    from paper_2502_01703_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    B.lib()    # fails loudly if the CUDA library is missing
    cfg = W.CONFIGS[WORKLOAD]
    n, P, d, bits = cfg["batch_rows"], cfg["P"], cfg["d"], cfg["bits"]
    rb = d * bits // 8
    off = W.task_offsets(TASKS).tolist()

    # ---- synthetic inputs, resident in HBM before the timed region ----
    g = W.student_t_gradients(n, P, seed=SEED + 100 * rank, device=dev, dtype=torch.bfloat16)
    m, v = W.adam_moments(P, seed=SEED + 1, device=dev)
    g_val = W.student_t_gradients(N_VAL, P, seed=SEED + 2, device=dev, dtype=torch.bfloat16)
    ws = torch.empty(B.qless_project_quantize_workspace(max(n, 256), P, d, bits), dtype=torch.uint8, device=dev)
    val_codes = torch.empty((1, N_VAL, rb), dtype=torch.uint8, device=dev)
    val_scales = torch.empty((1, N_VAL), dtype=torch.float32, device=dev)
    val_sumsq = torch.empty((1, N_VAL), dtype=torch.int32, device=dev)
    for r0 in range(0, N_VAL, 256):
        r1 = min(N_VAL, r0 + 256)
        B.qless_project_quantize(g_val[r0:r1], d, SEED, bits, workspace=ws,
                                 out=dict(codes=val_codes[0, r0:r1], scales=val_scales[0, r0:r1],
                                          sumsq=val_sumsq[0, r0:r1]))
    del g_val
    out = dict(codes=torch.empty((n, rb), dtype=torch.uint8, device=dev),
               scales=torch.empty(n, dtype=torch.float32, device=dev),
               sumsq=torch.empty(n, dtype=torch.int32, device=dev))
    scores = torch.empty(n, dtype=torch.float32, device=dev)
    indices = torch.empty(n, dtype=torch.int64, device=dev)
    ws_score = torch.empty(B.qless_score_workspace(n, N_VAL, 1, len(TASKS), d, bits), dtype=torch.uint8, device=dev)
    ws_sel = torch.empty(B.qless_select_topk_workspace(n), dtype=torch.uint8, device=dev)

    def step():
        B.qless_project_quantize(g, d, SEED, bits, m, v, out=out, workspace=ws)
        B.qless_score(out["codes"].unsqueeze(0), val_codes, out["scales"].unsqueeze(0), val_scales, [1.0], off,
                      d, bits, train_sumsq=out["sumsq"].unsqueeze(0), val_sumsq=val_sumsq, scores=scores,
                      workspace=ws_score)
        return B.qless_select_topk(scores, FRAC, indices=indices, workspace=ws_sel)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    B.qless_check()

    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    launches0 = B.qless_kernel_launches()
    B.qless_profile_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    prof = B.qless_profile_collect()
    B.qless_profile_enable(False)
    launches = B.qless_kernel_launches() - launches0
    B.qless_check()
    ms_total = max_over_ranks(ms_total, dist if world > 1 else None, dev)

    # ---- end to end through the host-buffer entry point (rank-local; host->device copies timed) ----
    e2e = None
    if not args.no_e2e:
        g_host = torch.empty((n, P), dtype=torch.bfloat16).pin_memory()
        g_host.copy_(g)
        host_out = dict(codes=torch.empty((n, rb), dtype=torch.uint8).pin_memory(),
                        scales=torch.empty(n, dtype=torch.float32).pin_memory(),
                        sumsq=torch.empty(n, dtype=torch.int32).pin_memory())
        idx_host = torch.empty(n, dtype=torch.int64).pin_memory()
        ws_host = torch.empty(B.qless_project_quantize_host_workspace(n, P, d, bits, B.BF16), dtype=torch.uint8, device=dev)
        del ws
        k_sel = int(FRAC * n + 1e-6)

        def step_e2e():
            B.qless_project_quantize_host(g_host, d, SEED, bits, m, v, out=host_out, workspace=ws_host, device=dev)
            out["codes"].copy_(host_out["codes"], non_blocking=True)
            out["scales"].copy_(host_out["scales"], non_blocking=True)
            out["sumsq"].copy_(host_out["sumsq"], non_blocking=True)
            B.qless_score(out["codes"].unsqueeze(0), val_codes, out["scales"].unsqueeze(0), val_scales, [1.0], off,
                          d, bits, train_sumsq=out["sumsq"].unsqueeze(0), val_sumsq=val_sumsq, scores=scores,
                          workspace=ws_score)
            sel = B.qless_select_topk(scores, FRAC, indices=indices, workspace=ws_sel)
            idx_host[:sel.numel()].copy_(sel, non_blocking=True)

        for _ in range(min(args.warmup, 2)):
            step_e2e()
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(args.e2e_steps):
            step_e2e()
        f1.record()
        barrier()
        ms_e2e = f0.elapsed_time(f1)
        ms_e2e = max_over_ranks(ms_e2e, dist if world > 1 else None, dev)
        h2d = n * P * 2 + n * rb + 2 * n * 4
        d2h = n * rb + 2 * n * 4 + k_sel * 8
        e2e = dict(value=whole_job_rate(n, args.e2e_steps, world, ms_e2e), unit="grads/s", h2d_bytes_per_step=h2d,
                   d2h_bytes_per_step=d2h, steps=args.e2e_steps, ms_per_step=ms_e2e / args.e2e_steps)
        # what bounds it: a plain pinned host-to-device copy of the same batch, nothing else running (outside the timed region)
        g.copy_(g_host, non_blocking=True)
        torch.cuda.synchronize()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        g.copy_(g_host, non_blocking=True)
        c1.record()
        torch.cuda.synchronize()
        e2e.update(plain_h2d_copy_ms=c0.elapsed_time(c1), plain_h2d_copy_gbs=n * P * 2 / c0.elapsed_time(c1) / 1e6)

    if rank == 0:
        peaks = load_peaks()
        value = whole_job_rate(n, args.steps, world, ms_total)
        proj_ms, proj_cnt = prof.get("project", (0.0, 0))
        flops = 2.0 * n * P * d
        achieved = flops / (proj_ms / max(proj_cnt, 1) * 1e-3) / 1e12 if proj_cnt else None
        roofline = roofline_entry(achieved, peaks, clocks, sm_count=torch.cuda.get_device_properties(dev).multi_processor_count)
        roofline.update(traffic=PROJECT_TRAFFIC_BYTES_PER_P * P, traffic_source=PROJECT_TRAFFIC_SOURCE,
                        flops_per_launch=flops, ms_per_launch=proj_ms / max(proj_cnt, 1))
        line = dict(metric="grads projected+quantized/s (P=2^23,d=8192)", value=value, unit="grads/s",
                    n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=ms_total / args.steps,
                    higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
                    config=bench_config(cfg),
                    clocks=clocks, gpu_launches=launches, roofline=roofline,
                    stages_ms_per_step={k: ms / args.steps for k, (ms, c) in prof.items()},
                    e2e=e2e)
        stages = None
        if world == 1 and not args.no_stages:
            del g, out
            torch.cuda.empty_cache()
            stages = stage_measurements(torch, B, W, dev, peaks)
            line["stages"] = stages
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline()
        if stages is not None:
            # the second half of the metric (train x validation scores per second per code width) and the HBM-bound
            # kernels, compact and last, so that a reader of the end of the line sees them
            line["summary"] = summarize(stages, line.get("cpu_baseline"), peaks, line["stages_ms_per_step"])
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-stages", action="store_true", help="skip the per-kernel measurements at their own sizes")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
