#!/usr/bin/env python
"""Benchmark of the scaled-array hot path on B200.

One step = one pass over every row of the hot path on synthetic, seeded inputs
shaped like GPT-style training tensors:
  1. scaled FP8 matmul 8192^3 (E4M3 x E4M3, fp32 accumulate) with fused AMAX, BF16 intermediate
  2. dynamic rescale pass 2: BF16 -> E4M3 with power-of-two rebalance
  H. the headline: 1 + 2 as ONE call, scalify_scaled_matmul(A, B, Y, AMAX, Yq): BF16 intermediate, fused AMAX and
     the E4M3 output written by the GEMM with the predicted power of two, confirmed (or rebuilt) by a check launch
  3. stand-alone dynamic rescale of a BF16 tensor (one read: the output is written with the predicted power of
     two while the statistic is gathered; a check launch repairs it if the prediction failed)
  4. scaled add of two BF16 tensors
  5. scaled LayerNorm forward  [131072, 1024] BF16
  6. scaled LayerNorm backward + L2 dynamic rescale of the input gradient to E5M2 (exact, in one pass: the
     gradient is written with the predicted power of two; a repair launch returns at once when it held)
  7. scaled Adam step over 125M parameters (E5M2 grads, FP16 scaled m/v/w)
Outside the step (own timed loop) the next-row variant is reported too: the same GEMM with delayed
rescaling - one kernel, E4M3 written directly with the previous step's statistic while this step's AMAX
is gathered, no BF16 intermediate, no pass 2.
`value` is the headline metric: 2*M*N*K / (time of call H), measured with CUDA events inside
the step.  Rows 3-7 are reported as GB/s of algorithmic bytes in `rows`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With --impl reference the fp64 CPU oracle is timed, as it stands, on a bounded sample of the
same workload on the host cores.
"""
import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "scaled FP8 GEMM+rescale TFLOP/s"
UNIT = "TFLOP/s"
N_GEMM = 8192
LN_R, LN_D = 131072, 1024
ADAM_N = 125_000_000
ADD_SHAPE = (8192, 8192)
ORACLE_SAMPLE_ROWS = 2048     # cpu_baseline leg: one sample (10-30 s of CPU work)
# --impl reference: the same 1024-row sample per timed step while the whole run stays within a few minutes
# (about 7 s per sample on 16 cores), fewer rows per step for longer runs
REFERENCE_ROWS_BUDGET = 24 * 1024

def gemm_dram_traffic():
    """DRAM bytes of one 8192^3 GEMM launch (dram__bytes_read.sum + dram__bytes_write.sum of an ncu capture) from
    the small record kept beside the profile summaries, or None when the kernel's source has changed since the
    capture was taken (the record carries a hash of the source files)."""
    import hashlib
    rec = os.path.join(ROOT, "profiles", "matmul_8192_dram_traffic.json")
    if not os.path.exists(rec):
        return None
    d = json.load(open(rec))
    h = hashlib.sha256()
    for f in d.get("sources", []):
        h.update(open(os.path.join(ROOT, f), "rb").read())
    return int(d["dram_bytes_per_launch"]) if h.hexdigest() == d.get("sources_sha256") else None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_burst=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only queries) every few milliseconds on a
    thread while the timed region runs."""

    def __init__(self, index, period_s=0.004):
        import threading
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self.err = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(vis.split(",")[index]) if vis and all(t.strip().isdigit() for t in vis.split(",")) else index
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # NVML missing: report it, do not fail the benchmark
            self.err = repr(e)
            return
        self.period = period_s
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self.nv
        bits = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(get_reasons(self.h))
                for name, bit in bits.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception as e:
                self.err = repr(e)
                break
            time.sleep(self.period)

    def mark(self):
        """Start of the timed region: what was sampled before (NVML start-up, warm-up) is dropped."""
        self.samples = []
        self.reasons = set()

    def stop(self):
        if self._thread is None:
            return dict(sm_mhz=None, sm_max_mhz=self.max_mhz, reasons=[f"unavailable: {self.err}"])
        self._stop.set()
        self._thread.join(timeout=2)
        if not self.samples:
            return dict(sm_mhz=None, sm_max_mhz=self.max_mhz, reasons=[f"no samples: {self.err}"])
        return dict(sm_mhz=statistics.median(self.samples), sm_min_mhz=min(self.samples),
                    sm_max_mhz=self.max_mhz, samples=len(self.samples), reasons=sorted(self.reasons))


def oracle_sample(rows):
    """One bounded sample of the headline workload on the oracle: `rows` output rows of the 8192^3 scaled
    matmul (BF16 intermediate) followed by the AMAX dynamic rescale of those rows to E4M3."""
    import oracle as orc
    import scalify_inputs as si
    c = oracle_sample.case
    if c is None:
        c = si.gemm_case(N_GEMM, "fwd", seed=1)
        oracle_sample.case = c
    t0 = time.perf_counter()
    Y, ys, _, _ = orc.scaled_matmul(c["A"][:rows], c["a_dtype"], c["a_scale"], c["Bt"], c["b_dtype"], c["b_scale"],
                                    orc.BF16, transB=True)
    orc.rescale(Y, orc.BF16, ys, orc.STAT_AMAX, orc.E4M3)
    dt = time.perf_counter() - t0
    return 2.0 * rows * N_GEMM * N_GEMM / dt / 1e12, dt


oracle_sample.case = None


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as orc
    rows = max(32, min(ORACLE_SAMPLE_ROWS, REFERENCE_ROWS_BUDGET // max(args.steps + min(args.warmup, 1), 1)))
    for _ in range(min(args.warmup, 1)):
        oracle_sample(rows)
    vals, times = [], []
    for _ in range(args.steps):
        v, dt = oracle_sample(rows)
        vals.append(v)
        times.append(dt)
    value = 2.0 * rows * N_GEMM * N_GEMM * len(times) / sum(times) / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"configs[1]: scaled GEMM M=N=K={N_GEMM} forward E4M3xE4M3 -> BF16 + AMAX rescale to E4M3"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                         "sample": f"{rows} of {N_GEMM} output rows of the 8192^3 GEMM + rescale of those rows per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def aggregate_over_ranks(dist, device, world, flops_per_rank, ms_per_step, head_ms, e2e_ms):
    """Replicas-only scaling: every rank runs the same step on its own GPU.  The job's time is the MAX over
    ranks of the device-measured times; the job's throughput is the work of all ranks over that time.
    `dist` is torch.distributed (initialised) or None for one process."""
    import torch
    if dist is not None:
        tt = torch.tensor([ms_per_step, head_ms, e2e_ms], device=device, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_per_step, head_ms, e2e_ms = [float(x) for x in tt]
    value = world * flops_per_rank / (head_ms * 1e-3) / 1e12
    e2e_value = world * flops_per_rank / (e2e_ms * 1e-3) / 1e12 if e2e_ms == e2e_ms else float("nan")
    return ms_per_step, head_ms, e2e_ms, value, e2e_value


def run_profile_row(args):
    """One row of the hot path alone, on a case that holds well under 2 GB on the device but is larger than
    L2, launched `--steps` times after `--warmup` launches.  Meant to be run under ncu."""
    import torch

    import paper_2407_17353_b200 as sc
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)

    def rnd(shape, dtype, tid, std=1.0):
        gen = torch.Generator(device=dev)
        gen.manual_seed(tid)
        return (torch.randn(shape, device=dev, dtype=torch.float32, generator=gen) * std).to(dtype)

    row = args.profile_row
    if row == "matmul":
        n = N_GEMM
        # --zero-operands: nothing toggles in the tensor cores' data path, so the 1000 W cap does not bind and the
        # SM clock stays up: the rate the kernel's structure allows (a diagnostic, not a benchmark value)
        std = 0.0 if args.zero_operands else 1.0
        A = sc.ScaledTensor.make(rnd((n, n), torch.float8_e4m3fn, 1, std), 1.0)
        Bt = sc.ScaledTensor.make(rnd((n, n), torch.float8_e4m3fn, 2, std), 2.0 ** -6)
        Y = sc.ScaledTensor.empty((n, n), torch.bfloat16, dev)
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, n, n), dev)
        fn = lambda t: sc.scalify_scaled_matmul(A, Bt, Y, ws, transB=True, stat=sc.STAT_AMAX)
        work = {"flop": 2.0 * n ** 3}
    elif row == "headline":
        n = N_GEMM
        A = sc.ScaledTensor.make(rnd((n, n), torch.float8_e4m3fn, 1), 1.0)
        Bt = sc.ScaledTensor.make(rnd((n, n), torch.float8_e4m3fn, 2), 2.0 ** -6)
        Y = sc.ScaledTensor.empty((n, n), torch.bfloat16, dev)
        Yq = sc.ScaledTensor.empty((n, n), torch.float8_e4m3fn, dev)
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, n, n), dev)
        fn = lambda t: sc.scalify_scaled_matmul(A, Bt, Y, ws, transB=True, stat=sc.STAT_AMAX, Yq=Yq)
        work = {"flop": 2.0 * n ** 3}
    elif row == "mx_quantize_t":
        n = N_GEMM
        Xa = sc.ScaledTensor.make(rnd((n, n), torch.bfloat16, 1), 1.0)
        Amt = sc.MxTensor(n, n, device=dev, transposed=True)
        fn = lambda t: sc.scalify_mx_quantize(Xa, Amt)
        work = {"bytes": n * n * (3.0 + 1.0 / 32)}
    elif row == "mx":
        n = N_GEMM
        Xa = sc.ScaledTensor.make(rnd((n, n), torch.bfloat16, 1), 1.0)
        Xb = sc.ScaledTensor.make(rnd((n, n), torch.bfloat16, 2), 1.0)
        Am, Bm = sc.MxTensor(n, n, device=dev), sc.MxTensor(n, n, device=dev)
        Y = sc.ScaledTensor.empty((n, n), torch.bfloat16, dev)
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, n, n), dev)

        def fn(t):
            sc.scalify_mx_quantize(Xa, Am)
            sc.scalify_mx_quantize(Xb, Bm)
            sc.scalify_mx_matmul(Am, Bm, Y, ws, stat=sc.STAT_AMAX)
        work = {"flop": 2.0 * n ** 3}
    elif row == "mx_gemm":
        # the block-scaled GEMM alone (operands quantised once, outside the timed calls); --zero-operands as above
        n = N_GEMM
        std = 0.0 if args.zero_operands else 1.0
        Xa = sc.ScaledTensor.make(rnd((n, n), torch.bfloat16, 1, std), 1.0)
        Xb = sc.ScaledTensor.make(rnd((n, n), torch.bfloat16, 2, std), 1.0)
        Am, Bm = sc.MxTensor(n, n, device=dev), sc.MxTensor(n, n, device=dev)
        sc.scalify_mx_quantize(Xa, Am)
        sc.scalify_mx_quantize(Xb, Bm)
        Y = sc.ScaledTensor.empty((n, n), torch.bfloat16, dev)
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, n, n), dev)
        fn = lambda t: sc.scalify_mx_matmul(Am, Bm, Y, ws, stat=sc.STAT_AMAX)
        work = {"flop": 2.0 * n ** 3}
    elif row == "attention":
        H, T, HD = 96, 1024, 64
        Qa, Ka, Va = (sc.ScaledTensor.make(rnd((H, T, HD), torch.float8_e4m3fn, 30 + i), 1.0) for i in range(3))
        Oa = sc.ScaledTensor.empty((H, T, HD), torch.bfloat16, dev)
        fn = lambda t: sc.scalify_scaled_attention(Qa, Ka, Va, Oa, sm_scale=0.125, causal=True)
        work = {"flop": 2.0 * H * T * T * HD}
    elif row == "attention_bwd":
        H, T, HD = 96, 1024, 64
        Qa, Ka, Va = (sc.ScaledTensor.make(rnd((H, T, HD), torch.float8_e4m3fn, 30 + i), 1.0) for i in range(3))
        Oa = sc.ScaledTensor.empty((H, T, HD), torch.bfloat16, dev)
        Pa = sc.ScaledTensor(torch.zeros((H, T, T), dtype=torch.uint8, device=dev).view(torch.float8_e4m3fn),
                             torch.ones(1, dtype=torch.float32, device=dev))
        sc.scalify_scaled_attention(Qa, Ka, Va, Oa, sm_scale=0.125, causal=True, P_dump=Pa)
        dOa = sc.ScaledTensor.make(rnd((H, T, HD), torch.float8_e5m2, 34), 2.0 ** -9)
        dSa = sc.ScaledTensor.empty((H, T, T), torch.float8_e5m2, dev)
        dQa, dKa, dVa = (sc.ScaledTensor.empty((H, T, HD), torch.bfloat16, dev) for _ in range(3))
        fn = lambda t: sc.scalify_scaled_attention_bwd(Qa, Ka, Va, Pa, dOa, dSa, dQa, dKa, dVa, sm_scale=0.125,
                                                       causal=True)
        work = {"flop": 4.0 * H * T * T * HD}
    elif row == "rescale":
        n = 8192 * 8192
        X = sc.ScaledTensor.make(rnd((n,), torch.bfloat16, 1, 37.0), 1.0)
        Yq = sc.ScaledTensor.empty((n,), torch.float8_e4m3fn, dev)
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, n), dev)
        fn = lambda t: sc.scalify_rescale(X, Yq, stat=sc.STAT_AMAX, ws=ws)
        work = {"bytes": 3.0 * n}   # read once, written once
    elif row == "add":
        n = 8192 * 8192
        P = sc.ScaledTensor.make(rnd((n,), torch.bfloat16, 1), 1.0)
        Q = sc.ScaledTensor.make(rnd((n,), torch.bfloat16, 2), 0.25)
        S = sc.ScaledTensor.empty((n,), torch.bfloat16, dev)
        fn = lambda t: sc.scalify_scaled_add(P, Q, S)
        work = {"bytes": 6.0 * n}
    elif row in ("layernorm", "layernorm_onepass"):
        R, d = 65536, 1024
        X = sc.ScaledTensor.make(rnd((R, d), torch.bfloat16, 3), 1.0)
        G = sc.ScaledTensor.make(rnd((R, d), torch.bfloat16, 4), 2.0 ** -10)
        gamma = sc.ScaledTensor.make((1.0 + 0.1 * rnd((d,), torch.float32, 5)).to(torch.bfloat16), 1.0)
        beta = sc.ScaledTensor.make(rnd((d,), torch.bfloat16, 6, 0.1), 1.0)
        LY = sc.ScaledTensor.empty((R, d), torch.bfloat16, dev)
        mean = torch.empty(R, dtype=torch.float32, device=dev)
        rinv = torch.empty(R, dtype=torch.float32, device=dev)
        dX = sc.ScaledTensor.empty((R, d), torch.bfloat16, dev)
        dXq = sc.ScaledTensor.empty((R, d), torch.float8_e5m2, dev)
        dg = sc.ScaledTensor.empty((d,), torch.float32, dev)
        db = sc.ScaledTensor.empty((d,), torch.float32, dev)
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d), dev)

        if row == "layernorm":
            def fn(t):
                sc.scalify_scaled_layernorm(X, gamma, beta, LY, eps=1e-5, mean=mean, rinv=rinv)
                sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, ws, eps=1e-5, stat_dx=sc.STAT_L2, dXq=dXq,
                                                dgamma=dg, dbeta=db)
            work = {"bytes": 13.0 * R * d}
        else:   # the backward with the exact rescale in one pass (dX = None)
            sc.scalify_scaled_layernorm(X, gamma, beta, LY, eps=1e-5, mean=mean, rinv=rinv)

            def fn(t):
                sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, None, ws, eps=1e-5, stat_dx=sc.STAT_L2,
                                                dXq=dXq, dgamma=dg, dbeta=db)
            work = {"bytes": 5.0 * R * d}
    else:
        n = 64 * 1024 * 1024
        ag = sc.ScaledTensor.make(rnd((n,), torch.float8_e5m2, 7), 2.0 ** -12)
        am = sc.ScaledTensor.make(rnd((n,), torch.float16, 8, 1.6), 2.0 ** -16)
        av = sc.ScaledTensor.make((rnd((n,), torch.float32, 9) ** 2).to(torch.float16), 2.0 ** -24)
        aw = sc.ScaledTensor.make(rnd((n,), torch.float16, 10, 1.28), 2.0 ** -6)
        adam = sc.AdamTensors([ag], [am], [av], [aw])
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, 1), dev)
        fn = lambda t: sc.scalify_scaled_adam_step(adam, ws, lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8,
                                                   step=1000 + (t % 2))
        work = {"bytes": 13.0 * n}
    for t in range(args.warmup):
        fn(t)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(args.steps):
        fn(t)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / max(args.steps, 1)
    out = {"profile_row": row, "ms_per_launch_group": ms}
    if "flop" in work:
        out["TFLOP/s"] = work["flop"] / (ms * 1e-3) / 1e12
    else:
        out["GB/s"] = work["bytes"] / (ms * 1e-3) / 1e9
    print(json.dumps(out))


def run_gpt_step(args):
    """Config 5: the GPT-2-small-shaped training step (12 layers, d 768, 12 heads, 8 x 1024 tokens, vocab 50257)
    composed from the C-ABI calls by the test harness (tests/gpt_model.py, unchecked here), launched call by
    call from Python or, with --graph, recorded once into a CUDA graph and replayed.  One JSON line."""
    import torch

    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import scalify_inputs as si
    from checked_ops import Ops
    from gpt_model import GPTConfig, ScaledGPT
    torch.cuda.set_device(0)
    cfg = GPTConfig()
    ops = Ops(check=False)
    model = ScaledGPT(cfg, ops, seed=6)
    n = cfg.batch * cfg.seq
    ids = torch.from_numpy(si.uniform_int(6, 901, (n,), cfg.vocab)).cuda()
    tgt = torch.from_numpy(si.uniform_int(6, 902, (n,), cfg.vocab)).cuda()
    for t in range(1, 1 + max(args.warmup, 1)):
        model.step(ids, tgt, t=t)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    calls = ops.calls
    if args.graph:
        stream = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                model.step(ids, tgt, t=10)
        calls = ops.calls - calls
        graph.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            graph.replay()
        e1.record()
    else:
        e0.record()
        for t in range(10, 10 + args.steps):
            model.step(ids, tgt, t=t)
        e1.record()
        calls = (ops.calls - calls) // max(args.steps, 1)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / max(args.steps, 1)
    print(json.dumps({"row": "config 5: GPT-2-small-shaped training step, all matmuls scaled FP8, FP16 scaled "
                             "optimizer state", "launch": "CUDA graph replay" if args.graph else "call by call from Python",
                      "ms_per_step": round(ms, 3), "tokens/s": round(n / ms * 1e3), "library_calls_per_step": calls}))


def run_hbm_sweep(args):
    """The HBM-bound rows at other sizes: LayerNorm forward / backward + rescale at R in {8192, 131072} and
    d in {768, 1024, 4096}; stand-alone rescale and add at 2^23, 2^26 and 2^28 elements.  Each case is
    launched back to back over a rotation of buffer sets larger than L2 in total (the small cases are
    L2- and launch-bound and say so).  One JSON line per case."""
    import torch

    import paper_2407_17353_b200 as sc
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peak = load_peaks()["hbm_gbs"]
    l2 = 126 * 2 ** 20

    def rnd(shape, dtype, tid):
        gen = torch.Generator(device=dev)
        gen.manual_seed(tid)
        return torch.randn(shape, device=dev, dtype=torch.float32, generator=gen).to(dtype)

    def timed(fns, iters):
        for f in fns:
            f()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fns[i % len(fns)]()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    def report(name, ms, nbytes, sets, footprint):
        gbs = nbytes / (ms * 1e-3) / 1e9
        print(json.dumps({"sweep": name, "ms": round(ms, 4), "GB/s": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peak, 3),
                          "buffer_sets": sets, "note": "larger than L2 per launch" if footprint > l2 else
                          "fits L2: rotation over %d sets makes the inputs cold, the launch itself is short" % sets}))

    iters = max(10, args.steps)
    for R in (8192, 131072):
        for d in (768, 1024, 4096):
            per_set = R * d * 2 * 4
            sets = max(1, min(8, -(-2 * l2 // per_set)))
            fw, bw, bwd_delayed, bwd_onepass = [], [], [], []
            gamma = sc.ScaledTensor.make(torch.ones(d, device=dev).to(torch.bfloat16), 1.0)
            beta = sc.ScaledTensor.make(torch.zeros(d, device=dev).to(torch.bfloat16), 1.0)
            ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d), dev)
            ws1 = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, R, d), dev)   # keeps the prediction
            for k in range(sets):
                X = sc.ScaledTensor.make(rnd((R, d), torch.bfloat16, 10 + k), 1.0)
                G = sc.ScaledTensor.make(rnd((R, d), torch.bfloat16, 20 + k), 2.0 ** -10)
                Y = sc.ScaledTensor.empty((R, d), torch.bfloat16, dev)
                dX = sc.ScaledTensor.empty((R, d), torch.bfloat16, dev)
                dXq = sc.ScaledTensor.empty((R, d), torch.float8_e5m2, dev)
                dg = sc.ScaledTensor.empty((d,), torch.float32, dev)
                db = sc.ScaledTensor.empty((d,), torch.float32, dev)
                mean = torch.empty(R, dtype=torch.float32, device=dev)
                rinv = torch.empty(R, dtype=torch.float32, device=dev)
                fw.append(lambda X=X, Y=Y, mean=mean, rinv=rinv: sc.scalify_scaled_layernorm(
                    X, gamma, beta, Y, eps=1e-5, mean=mean, rinv=rinv))
                bw.append(lambda G=G, X=X, mean=mean, rinv=rinv, dX=dX, dXq=dXq, dg=dg, db=db:
                          sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, ws, eps=1e-5, stat_dx=sc.STAT_L2,
                                                          dXq=dXq, dgamma=dg, dbeta=db))
                bwd_delayed.append(lambda G=G, X=X, mean=mean, rinv=rinv, dXq=dXq, dg=dg, db=db:
                                   sc.scalify_scaled_layernorm_bwd_delayed(G, X, gamma, mean, rinv, ws.statistic(), dXq, ws,
                                                                           eps=1e-5, stat_dx=sc.STAT_L2, dgamma=dg,
                                                                           dbeta=db))
                bwd_onepass.append(lambda G=G, X=X, mean=mean, rinv=rinv, dXq=dXq, dg=dg, db=db:
                                   sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, None, ws1, eps=1e-5,
                                                                   stat_dx=sc.STAT_L2, dXq=dXq, dgamma=dg, dbeta=db))
            report(f"LayerNorm fwd {R}x{d} BF16->BF16", timed(fw, iters), R * d * 4 + R * 8, sets, R * d * 4)
            report(f"LayerNorm bwd + L2 rescale to E5M2 {R}x{d}", timed(bw, iters), R * d * 9 + R * 8, sets, R * d * 6)
            report(f"LayerNorm bwd, delayed L2 rescale, E5M2 out in one pass {R}x{d}", timed(bwd_delayed, iters),
                   R * d * 5 + R * 8, sets, R * d * 5)
            report(f"LayerNorm bwd + exact L2 rescale to E5M2 in one pass (dX = NULL) {R}x{d}", timed(bwd_onepass, iters),
                   R * d * 5 + R * 8, sets, R * d * 5)
            del fw, bw, bwd_delayed, bwd_onepass
            torch.cuda.empty_cache()
    for lg in (23, 26, 28):
        n = 1 << lg
        sets = max(1, min(8, -(-2 * l2 // (n * 3))))
        rs, ad = [], []
        ws = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, n), dev)
        for k in range(sets):
            X = sc.ScaledTensor.make(rnd((n,), torch.bfloat16, 30 + k), 1.0)
            Z = sc.ScaledTensor.make(rnd((n,), torch.bfloat16, 40 + k), 0.25)
            Yq = sc.ScaledTensor.empty((n,), torch.float8_e4m3fn, dev)
            S = sc.ScaledTensor.empty((n,), torch.bfloat16, dev)
            rs.append(lambda X=X, Yq=Yq: sc.scalify_rescale(X, Yq, stat=sc.STAT_AMAX, ws=ws))
            ad.append(lambda X=X, Z=Z, S=S: sc.scalify_scaled_add(X, Z, S))
        report(f"stand-alone dynamic rescale BF16->E4M3 2^{lg} elements (one read)", timed(rs, iters), 3 * n, sets, 3 * n)
        report(f"scaled add BF16 2^{lg} elements", timed(ad, iters), 6 * n, sets, 6 * n)
        del rs, ad
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (for ncu launch lists)")
    ap.add_argument("--hbm-sweep", action="store_true",
                    help="print one JSON line per size of the HBM-bound rows (LayerNorm, rescale, add) instead of the step")
    ap.add_argument("--no-next", action="store_true",
                    help="skip the separately timed next-row variants f1, f2 (for ncu launch lists of the step)")
    ap.add_argument("--profile-row", default=None, choices=["matmul", "headline", "mx", "mx_gemm", "mx_quantize_t", "attention", "attention_bwd", "rescale", "add", "layernorm",
                             "layernorm_onepass", "adam"],
                    help="run only this row on a reduced, still larger-than-L2 case (for ncu captures)")
    ap.add_argument("--gpt-step", action="store_true",
                    help="time the config-5 step (GPT-2-small shapes) instead; with --graph replayed from a CUDA graph")
    ap.add_argument("--graph", action="store_true")
    ap.add_argument("--zero-operands", action="store_true",
                    help="with --profile-row matmul or mx_gemm: all-zero operands (the kernel without the power cap binding)")
    args = ap.parse_args()
    if args.gpt_step:
        run_gpt_step(args)
        return
    if args.impl == "reference":
        run_reference(args)
        return
    if args.hbm_sweep:
        run_hbm_sweep(args)
        return
    if args.profile_row:
        run_profile_row(args)
        return

    import numpy as np
    import torch

    import paper_2407_17353_b200 as sc
    import scalify_inputs as si

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()
    W = max(args.warmup, 3)
    K = args.steps

    def dev_bits(bits, code):
        b = np.ascontiguousarray(bits)
        t = torch.from_numpy(b.view({1: np.int8, 2: np.int16, 4: np.int32}[b.dtype.itemsize])).to(dev)
        return t.view(sc.TORCH_DTYPE[code])

    # ------------------------------------------------------------------ inputs (seeded, synthetic)
    seed = 1 + rank
    g = si.gemm_case(N_GEMM, "fwd", seed=seed)
    hA = torch.from_numpy(g["A"].view(np.int8)).pin_memory()
    hB = torch.from_numpy(g["Bt"].view(np.int8)).pin_memory()
    A = sc.ScaledTensor.make(dev_bits(g["A"], si.E4M3), g["a_scale"])
    Bt = sc.ScaledTensor.make(dev_bits(g["Bt"], si.E4M3), g["b_scale"])
    Y = sc.ScaledTensor.empty((N_GEMM, N_GEMM), torch.bfloat16, dev)
    Yq = sc.ScaledTensor.empty((N_GEMM, N_GEMM), torch.float8_e4m3fn, dev)
    ws_mm = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, N_GEMM, N_GEMM), dev)

    def rnd(shape, dtype, tid, std=1.0):
        gen = torch.Generator(device=dev)
        gen.manual_seed(1000 * seed + tid)
        return (torch.randn(shape, device=dev, dtype=torch.float32, generator=gen) * std).to(dtype)

    # rows 3/4: BF16 tensors of the GEMM-output size
    P = sc.ScaledTensor.make(rnd(ADD_SHAPE, torch.bfloat16, 1), 1.0)
    Q = sc.ScaledTensor.make(rnd(ADD_SHAPE, torch.bfloat16, 2), 2.0 ** -2)
    S = sc.ScaledTensor.empty(ADD_SHAPE, torch.bfloat16, dev)
    Rq = sc.ScaledTensor.empty(ADD_SHAPE, torch.float8_e4m3fn, dev)
    ws_rs = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_RESCALE, ADD_SHAPE[0] * ADD_SHAPE[1]), dev)
    # rows 5/6: LayerNorm
    X = sc.ScaledTensor.make(rnd((LN_R, LN_D), torch.bfloat16, 3), 1.0)
    G = sc.ScaledTensor.make(rnd((LN_R, LN_D), torch.bfloat16, 4), 2.0 ** -10)
    gamma = sc.ScaledTensor.make((1.0 + 0.1 * rnd((LN_D,), torch.float32, 5)).to(torch.bfloat16), 1.0)
    beta = sc.ScaledTensor.make(rnd((LN_D,), torch.bfloat16, 6, 0.1), 1.0)
    LY = sc.ScaledTensor.empty((LN_R, LN_D), torch.bfloat16, dev)
    mean = torch.empty(LN_R, dtype=torch.float32, device=dev)
    rinv = torch.empty(LN_R, dtype=torch.float32, device=dev)
    dX = sc.ScaledTensor.empty((LN_R, LN_D), torch.bfloat16, dev)
    dXq = sc.ScaledTensor.empty((LN_R, LN_D), torch.float8_e5m2, dev)
    dg = sc.ScaledTensor.empty((LN_D,), torch.float32, dev)
    db = sc.ScaledTensor.empty((LN_D,), torch.float32, dev)
    ws_ln = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, LN_R, LN_D), dev)
    # row 7: Adam (one flat tensor of 125M parameters; state is re-seeded from copies so it stays in range)
    ag = sc.ScaledTensor.make(rnd((ADAM_N,), torch.float8_e5m2, 7), 2.0 ** -12)
    am0 = rnd((ADAM_N,), torch.float16, 8, 1.6)
    av0 = (rnd((ADAM_N,), torch.float32, 9) ** 2).to(torch.float16)
    aw0 = rnd((ADAM_N,), torch.float16, 10, 1.28)
    am = sc.ScaledTensor.make(am0.clone(), 2.0 ** -16)
    av = sc.ScaledTensor.make(av0.clone(), 2.0 ** -24)
    aw = sc.ScaledTensor.make(aw0.clone(), 2.0 ** -6)
    adam = sc.AdamTensors([ag], [am], [av], [aw])
    ws_ad = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_ADAM, 1), dev)
    del am0, av0, aw0

    Yd = sc.ScaledTensor.empty((N_GEMM, N_GEMM), torch.float8_e4m3fn, dev)
    stat_state = torch.full((1,), 4.0, dtype=torch.float32, device=dev)

    Yq2 = sc.ScaledTensor.empty((N_GEMM, N_GEMM), torch.float8_e4m3fn, dev)
    ws_head = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, N_GEMM, N_GEMM), dev)   # keeps the prediction
    n_ev = 9
    # kernels of this library per step: headline call (matmul + check launch), one-read rescale (statistic with the
    # predicted output + check launch), add, LayerNorm fwd, LayerNorm bwd + finalize + repair launch, Adam scales +
    # update
    launches_per_step = 2 + 2 + 1 + 1 + 3 + 2
    ws_ln1 = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_LAYERNORM_BWD, LN_R, LN_D), dev)   # keeps the prediction
    dXq1 = sc.ScaledTensor.empty((LN_R, LN_D), torch.float8_e5m2, dev)

    def step(t, evs=None, form=0):
        """form 0: the headline as one call and the LayerNorm gradient's rescale in one pass; 1: the same work as two
        calls (GEMM + AMAX, then pass 2, each with a time of its own) and the LayerNorm backward with its stored BF16
        intermediate and a second pass; 2: the one call without the BF16 intermediate (Y = NULL)."""
        def mark(i):
            if evs is not None:
                evs[i].record()
        mark(0)
        if form == 1:
            sc.scalify_scaled_matmul(A, Bt, Y, ws_mm, transB=True, stat=sc.STAT_AMAX, Yq=None)
            mark(1)
            sc.scalify_rescale(Y, Yq, stat=sc.STAT_AMAX, stat_in=ws_mm.statistic())
        else:
            # GEMM + fused AMAX + rescale to E4M3 as ONE call of the library's main entry point
            sc.scalify_scaled_matmul(A, Bt, None if form == 2 else Y, ws_head, transB=True, stat=sc.STAT_AMAX, Yq=Yq2)
            mark(1)
        mark(2)
        sc.scalify_rescale(P, Rq, stat=sc.STAT_AMAX, ws=ws_rs)
        mark(3)
        sc.scalify_scaled_add(P, Q, S)
        mark(4)
        sc.scalify_scaled_layernorm(X, gamma, beta, LY, eps=1e-5, mean=mean, rinv=rinv)
        mark(5)
        if form == 1:
            sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, dX, ws_ln, eps=1e-5, stat_dx=sc.STAT_L2, dXq=dXq,
                                            dgamma=dg, dbeta=db)
        else:
            # a6 in ONE pass (dX = None): the exact dynamic rescale with the predicted power of two
            sc.scalify_scaled_layernorm_bwd(G, X, gamma, mean, rinv, None, ws_ln1, eps=1e-5, stat_dx=sc.STAT_L2,
                                            dXq=dXq1, dgamma=dg, dbeta=db)
        mark(6)
        sc.scalify_scaled_adam_step(adam, ws_ad, lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8, step=1000 + t)
        mark(7)
        mark(8)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def graph_ms(calls, n_calls):
        """Average device time per call of `n_calls` library calls (round robin over `calls`) recorded once
        into a CUDA graph and replayed: what a launch-bound call costs on the device once Python and the
        driver's launch path are out of the way."""
        side = torch.cuda.Stream(dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for f in calls:
                f()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(n_calls):
                    calls[i % len(calls)]()
        torch.cuda.current_stream().wait_stream(side)
        g.replay()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(3):
            g.replay()
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1) / (3 * n_calls)
        del g
        return ms

    # the sampler thread starts before the warm-up, so that NVML's start-up is over when the timed region begins
    sampler = ClockSampler(local_rank) if rank == 0 else None
    for t in range(W):
        step(t, None)
    barrier()
    for w in (ws_mm, ws_head, ws_rs, ws_ln, ws_ln1, ws_ad):
        st = w.check_status()
        if st != 0:
            raise SystemExit(f"device status {st} after warm-up")

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(K)]
    barrier()
    if sampler is not None:
        sampler.mark()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for t in range(K):
        step(W + t, evs[t])
    t_end.record()
    barrier()
    clocks = sampler.stop() if sampler is not None else None
    total_ms = t_start.elapsed_time(t_end)
    seg = np.array([[evs[t][i].elapsed_time(evs[t][i + 1]) for i in range(n_ev - 1)] for t in range(K)])
    seg_ms = seg.mean(axis=0)
    for w in (ws_mm, ws_head, ws_rs, ws_ln, ws_ln1, ws_ad):
        st = w.check_status()
        if st & sc.DEV_TIMEOUT:
            raise SystemExit(f"device status {st} in the timed region")

    # The same step twice more: with the headline's work as TWO calls (the GEMM with fused AMAX and the rebalance
    # pass each get a time of their own, in the same surroundings), and with the one call in its FP8-only form
    # (Y = NULL).  All three forms must leave the same E4M3 output and scale, bit for bit.
    two_call_ms = [float("nan"), float("nan")]
    ln_two_pass_ms = float("nan")
    fp8_only_ms = float("nan")
    if not args.no_next:
        for form in (1, 2):
            for t in range(3):
                step(W + K + t, None, form)
            barrier()
            evs2 = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(K)]
            for t in range(K):
                step(W + K + 3 + t, evs2[t], form)
            barrier()
            if form == 1:
                two_call_ms = [float(np.mean([evs2[t][0].elapsed_time(evs2[t][1]) for t in range(K)])),
                               float(np.mean([evs2[t][1].elapsed_time(evs2[t][2]) for t in range(K)]))]
                ln_two_pass_ms = float(np.mean([evs2[t][5].elapsed_time(evs2[t][6]) for t in range(K)]))
                same = torch.equal(Yq.data.view(torch.uint8), Yq2.data.view(torch.uint8)) and \
                    float(Yq.scale.item()) == float(Yq2.scale.item())
                if not same:
                    raise SystemExit("the one-call headline and the two-call form disagree")
                same_ln = torch.equal(dXq.data.view(torch.uint8), dXq1.data.view(torch.uint8)) and \
                    dXq.scale_value() == dXq1.scale_value() and \
                    torch.equal(ws_ln.statistic().view(torch.int32), ws_ln1.statistic().view(torch.int32))
                if not same_ln:
                    raise SystemExit("the one-pass LayerNorm gradient rescale and the two-pass form disagree")
            else:
                fp8_only_ms = float(np.mean([evs2[t][0].elapsed_time(evs2[t][2]) for t in range(K)]))
                if not torch.equal(Yq.data.view(torch.uint8), Yq2.data.view(torch.uint8)):
                    raise SystemExit("the FP8-only headline form and the two-call form disagree")

    flops = 2.0 * N_GEMM ** 3
    head_ms = float(seg_ms[0])
    value_local = flops / (head_ms * 1e-3) / 1e12
    ms_per_step = total_ms / K

    # ------------------------------------------------------------------ next-row variant, timed on its own
    def delayed_step():
        sc.scalify_scaled_matmul_delayed(A, Bt, stat_state, Yd, ws_mm, transB=True, stat=sc.STAT_AMAX,
                                         stat_out=stat_state)
    for _ in range(0 if args.no_next else 3):
        delayed_step()
    barrier()
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d_iters = 0 if args.no_next else max(3, min(K, 20))
    d0.record()
    for _ in range(d_iters):
        delayed_step()
    d1.record()
    barrier()
    delayed_ms = d0.elapsed_time(d1) / d_iters if d_iters else float("nan")

    # LayerNorm backward with delayed rescale: E5M2 gradient in one pass with the previous step's statistic,
    # this step's statistic left in the same word (5 B/elem instead of 9)
    ln_stat = ws_ln.statistic()

    def ln_delayed_step():
        sc.scalify_scaled_layernorm_bwd_delayed(G, X, gamma, mean, rinv, ln_stat, dXq, ws_ln, eps=1e-5,
                                                stat_dx=sc.STAT_L2, dgamma=dg, dbeta=db)
    for _ in range(0 if args.no_next else 3):
        ln_delayed_step()
    barrier()
    l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l_iters = 0 if args.no_next else max(3, min(K, 20))
    l0.record()
    for _ in range(l_iters):
        ln_delayed_step()
    l1.record()
    barrier()
    ln_delayed_ms = l0.elapsed_time(l1) / l_iters if l_iters else float("nan")

    # Adam that also writes the E4M3 compute copy of the updated weight (1 more byte per parameter)
    awc = sc.ScaledTensor.make(torch.empty(ADAM_N, dtype=torch.float8_e4m3fn, device=dev), 1.0)

    wc_list = [awc]  # the same list object every call, so the descriptors are marshalled once

    def adam_cast_step(t):
        sc.scalify_scaled_adam_step_cast(adam, wc_list, ws_ad, lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8,
                                         step=2000 + t)
    for t in range(0 if args.no_next else 3):
        adam_cast_step(t)
    barrier()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c_iters = 0 if args.no_next else max(3, min(K, 20))
    c0.record()
    for t in range(c_iters):
        adam_cast_step(t)
    c1.record()
    barrier()
    adam_cast_ms = c0.elapsed_time(c1) / c_iters if c_iters else float("nan")

    # Block-scaled variant (E8M0 exponent per 32 elements of K): quantise both BF16 operands, then the
    # block-scaled GEMM with fused AMAX, BF16 out
    mx_q_ms = mx_mm_ms = mx_qt_ms = mx_mmt_ms = float("nan")
    if not args.no_next:
        Xa = sc.ScaledTensor.make(rnd((N_GEMM, N_GEMM), torch.bfloat16, 21), 1.0)
        Xb = sc.ScaledTensor.make(rnd((N_GEMM, N_GEMM), torch.bfloat16, 22), 1.0)
        Am, Bm = sc.MxTensor(N_GEMM, N_GEMM, device=dev), sc.MxTensor(N_GEMM, N_GEMM, device=dev)

        def mx_quant():
            sc.scalify_mx_quantize(Xa, Am)
            sc.scalify_mx_quantize(Xb, Bm)

        def mx_mm():
            sc.scalify_mx_matmul(Am, Bm, Y, ws_mm, stat=sc.STAT_AMAX)

        # the weight-gradient form: both operands stored with the contraction axis slow ([K, rows])
        Amt, Bmt = (sc.MxTensor(N_GEMM, N_GEMM, device=dev, transposed=True) for _ in range(2))

        def mx_quant_t():
            sc.scalify_mx_quantize(Xa, Amt)
            sc.scalify_mx_quantize(Xb, Bmt)

        def mx_mm_t():
            sc.scalify_mx_matmul(Amt, Bmt, Y, ws_mm, stat=sc.STAT_AMAX)
        x_iters = max(3, min(K, 20))
        times = []
        for fn in (mx_quant, mx_mm, mx_quant_t, mx_mm_t):
            for _ in range(3):
                fn()
            barrier()
            x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            x0.record()
            for _ in range(x_iters):
                fn()
            x1.record()
            barrier()
            times.append(x0.elapsed_time(x1) / x_iters)
        mx_q_ms, mx_mm_ms, mx_qt_ms, mx_mmt_ms = times
        del Xa, Xb, Am, Bm, Amt, Bmt

    # Fused attention forward on the config-5 shape: 8 sequences x 12 heads, 1024 tokens, head dimension 64
    att_ms = att_bwd_ms = att_graph_ms = att_bwd_graph_ms = float("nan")
    ATT_H, ATT_T, ATT_HD = 96, 1024, 64
    ATT_SETS = 9   # 9 x 31 MB of Q, K, V, O: twice the L2, so no call finds its inputs there
    if not args.no_next:
        att_sets = []
        for k in range(ATT_SETS):
            q_, k_, v_ = (sc.ScaledTensor.make(rnd((ATT_H, ATT_T, ATT_HD), torch.float8_e4m3fn, 30 + i + 3 * k), 1.0)
                          for i in range(3))
            att_sets.append((q_, k_, v_, sc.ScaledTensor.empty((ATT_H, ATT_T, ATT_HD), torch.bfloat16, dev)))
        att_calls = [lambda t=t: sc.scalify_scaled_attention(t[0], t[1], t[2], t[3], sm_scale=0.125, causal=True)
                     for t in att_sets]
        Qa, Ka, Va, Oa = att_sets[0]
        for f in att_calls:
            f()
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_iters = max(ATT_SETS, min(K, 2 * ATT_SETS))
        a0.record()
        for i in range(a_iters):
            att_calls[i % ATT_SETS]()
        a1.record()
        barrier()
        att_ms = a0.elapsed_time(a1) / a_iters
        att_graph_ms = graph_ms(att_calls, 2 * ATT_SETS)
        # ... and its backward (two launches): P from the forward's copy, dO as E5M2
        Pa = sc.ScaledTensor(torch.zeros((ATT_H, ATT_T, ATT_T), dtype=torch.uint8, device=dev).view(torch.float8_e4m3fn),
                             torch.ones(1, dtype=torch.float32, device=dev))
        sc.scalify_scaled_attention(Qa, Ka, Va, Oa, sm_scale=0.125, causal=True, P_dump=Pa)
        dOa = sc.ScaledTensor.make(rnd((ATT_H, ATT_T, ATT_HD), torch.float8_e5m2, 34), 2.0 ** -9)
        dSa = sc.ScaledTensor.empty((ATT_H, ATT_T, ATT_T), torch.float8_e5m2, dev)
        dQa, dKa, dVa = (sc.ScaledTensor.empty((ATT_H, ATT_T, ATT_HD), torch.bfloat16, dev) for _ in range(3))
        att_bwd = lambda: sc.scalify_scaled_attention_bwd(Qa, Ka, Va, Pa, dOa, dSa, dQa, dKa, dVa, sm_scale=0.125,
                                                          causal=True)
        for _ in range(3):
            att_bwd()
        barrier()
        a0.record()
        for _ in range(a_iters):
            att_bwd()
        a1.record()
        barrier()
        att_bwd_ms = a0.elapsed_time(a1) / a_iters
        att_bwd_graph_ms = graph_ms([att_bwd], 10)   # P and dS are 100 MB each: larger than the L2 by themselves
        del Qa, Ka, Va, Oa, Pa, dOa, dSa, dQa, dKa, dVa, att_sets, att_calls

    # ------------------------------------------------------------------ configs[1]: the other sizes and formats
    # M = N = K in {1024, 4096, 8192}, forward E4M3 x E4M3 and gradient E5M2 x E4M3, each as the one-call form
    # (BF16 intermediate + fused AMAX + E4M3 output), back to back over a rotation of buffer sets that together
    # exceed twice the L2 (one workspace per set, so that every set keeps its own prediction)
    sweep_rows = []
    if not args.no_next:
        l2 = 126 * 2 ** 20
        for n in (1024, 4096, N_GEMM):
            for kind, a_dt, a_s in (("forward E4M3 x E4M3", torch.float8_e4m3fn, 1.0),
                                    ("gradient E5M2 x E4M3", torch.float8_e5m2, 2.0 ** -10)):
                per_set = n * n * 5
                sets = max(2, min(64, -(-2 * l2 // per_set)))
                calls = []
                for k in range(sets):
                    As = sc.ScaledTensor.make(rnd((n, n), a_dt, 50 + 2 * k), a_s)
                    Bs = sc.ScaledTensor.make(rnd((n, n), torch.float8_e4m3fn, 51 + 2 * k), 2.0 ** -6)
                    Ys = sc.ScaledTensor.empty((n, n), torch.bfloat16, dev)
                    Yqs_ = sc.ScaledTensor.empty((n, n), torch.float8_e4m3fn, dev)
                    wss = sc.Workspace(sc.scalify_workspace_bytes(sc.OP_MATMUL, n, n), dev)
                    calls.append(lambda As=As, Bs=Bs, Ys=Ys, Yqs_=Yqs_, wss=wss: sc.scalify_scaled_matmul(
                        As, Bs, Ys, wss, transB=True, stat=sc.STAT_AMAX, Yq=Yqs_))
                for _ in range(2):
                    for f in calls:
                        f()
                barrier()
                g_iters = max(len(calls), min(K, 20)) if n == N_GEMM else 4 * len(calls)
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record()
                for i in range(g_iters):
                    calls[i % len(calls)]()
                g1.record()
                barrier()
                g_ms = g0.elapsed_time(g1) / g_iters
                sweep = {"row": f"configs[1] {kind}, M=N=K={n}: GEMM + fused AMAX + rescale to E4M3, one call "
                                f"(own loop, back to back over {sets} buffer sets)",
                         "ms": round(g_ms, 4), "TFLOP/s": round(2.0 * n ** 3 / (g_ms * 1e-3) / 1e12, 1)}
                if n < N_GEMM:
                    # a call this short is bound by the launch path from Python; the same calls replayed from a CUDA graph
                    gg_ms = graph_ms(calls, 2 * len(calls))
                    sweep["ms_cuda_graph"] = round(gg_ms, 4)
                    sweep["TFLOP/s_cuda_graph"] = round(2.0 * n ** 3 / (gg_ms * 1e-3) / 1e12, 1)
                sweep_rows.append(sweep)
                del calls
                torch.cuda.empty_cache()

    # ------------------------------------------------------------------ end to end through host buffers
    hY = torch.empty((N_GEMM, N_GEMM), dtype=torch.int8).pin_memory()
    hscale = torch.empty(1, dtype=torch.float32).pin_memory()
    # Two sets of device buffers and three streams (copy in, compute, copy out): step i's host->device
    # copies, step i-1's kernels and step i-2's device->host copies run at the same time.  Every step
    # still copies its own inputs in and its own result out inside the timed region.
    DEPTH = 2
    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    dAs = [torch.empty((N_GEMM, N_GEMM), dtype=torch.int8, device=dev) for _ in range(DEPTH)]
    dBs = [torch.empty((N_GEMM, N_GEMM), dtype=torch.int8, device=dev) for _ in range(DEPTH)]
    A2s = [sc.ScaledTensor(t.view(torch.float8_e4m3fn), A.scale) for t in dAs]
    B2s = [sc.ScaledTensor(t.view(torch.float8_e4m3fn), Bt.scale) for t in dBs]
    Yqs = [sc.ScaledTensor.empty((N_GEMM, N_GEMM), torch.float8_e4m3fn, dev) for _ in range(DEPTH)]
    ev_in = [torch.cuda.Event() for _ in range(DEPTH)]
    ev_cmp = [torch.cuda.Event() for _ in range(DEPTH)]
    ev_out = [torch.cuda.Event() for _ in range(DEPTH)]
    e2e_count = [0]

    def e2e_step():
        i = e2e_count[0]
        b = i % DEPTH
        e2e_count[0] = i + 1
        with torch.cuda.stream(s_in):
            if i >= DEPTH:
                s_in.wait_event(ev_cmp[b])  # the kernels that read this buffer set have finished
            dAs[b].copy_(hA, non_blocking=True)
            dBs[b].copy_(hB, non_blocking=True)
            ev_in[b].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(ev_in[b])
            if i >= DEPTH:
                s_cmp.wait_event(ev_out[b])  # the previous result in this set has been read out
            sc.scalify_scaled_matmul(A2s[b], B2s[b], Y, ws_mm, transB=True, stat=sc.STAT_AMAX, Yq=Yqs[b])
            ev_cmp[b].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[b])
            hY.copy_(Yqs[b].data.view(torch.int8), non_blocking=True)
            hscale.copy_(Yqs[b].scale, non_blocking=True)
            ev_out[b].record(s_out)

    def e2e_join():
        cur = torch.cuda.current_stream(dev)
        for s_ in (s_in, s_cmp, s_out):
            cur.wait_stream(s_)

    e2e_iters = 0 if args.no_e2e else max(6, min(K, 20))
    for s_ in (s_in, s_cmp, s_out):
        s_.wait_stream(torch.cuda.current_stream(dev))
    for _ in range(3 if e2e_iters else 0):
        e2e_step()
    e2e_join()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s_ in (s_in, s_cmp, s_out):
        s_.wait_stream(torch.cuda.current_stream(dev))
    for _ in range(e2e_iters):
        e2e_step()
    e2e_join()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / max(e2e_iters, 1) if e2e_iters else float('nan')
    e2e_local = flops / (e2e_ms * 1e-3) / 1e12

    # ------------------------------------------------------------------ reduce over ranks (max time)
    ms_per_step, head_ms_max, e2e_ms_max, value, e2e_value = aggregate_over_ranks(
        dist, dev, world, flops, ms_per_step, head_ms, e2e_ms)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    n_add = ADD_SHAPE[0] * ADD_SHAPE[1]
    n_ln = LN_R * LN_D
    hbm = peaks["hbm_gbs"]

    def row(name, ms, nbytes):
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"row": name, "ms": round(float(ms), 4), "GB/s": round(gbs, 1), "frac_of_hbm_peak": round(gbs / hbm, 3)}

    rows = [
        {"row": "HEADLINE a1+a2+a3 as one call: scalify_scaled_matmul(A, B, Y, AMAX, Yq) - BF16 intermediate, fused "
                "AMAX, E4M3 written by the GEMM with the predicted power of two, check launch (bit-identical to the "
                "two calls)", "ms": round(float(seg_ms[0]), 4), "TFLOP/s": round(flops / (seg_ms[0] * 1e-3) / 1e12, 1)},
        {"row": "a1+a2 scaled FP8 matmul 8192^3 + fused AMAX alone (second pass of the same step, two-call form)",
         "ms": round(two_call_ms[0], 4), "TFLOP/s": round(flops / (two_call_ms[0] * 1e-3) / 1e12, 1)},
        row("a3 rescale pass 2 BF16->E4M3 alone (second pass of the same step, 3 B/elem)", two_call_ms[1],
            3 * N_GEMM * N_GEMM),
        {"row": "a1+a2+a3 as two calls (second pass of the same step)", "ms": round(two_call_ms[0] + two_call_ms[1], 4),
         "TFLOP/s": round(flops / ((two_call_ms[0] + two_call_ms[1]) * 1e-3) / 1e12, 1)},
        dict(row("a3'+a3 stand-alone dynamic rescale BF16->E4M3, one read: output written with the predicted power of "
                 "two while the statistic is gathered, check launch (3 B/elem; two reads, 5 B/elem, before)", seg_ms[2],
                 3 * n_add), GBps_at_5_bytes_per_elem=round(5 * n_add / (seg_ms[2] * 1e-3) / 1e9, 1)),
        row("a4 scaled add BF16 (6 B/elem)", seg_ms[3], 6 * n_add),
        row("a5 scaled LayerNorm fwd BF16->BF16 (4 B/elem + 8 B/row)", seg_ms[4], 4 * n_ln + 8 * LN_R),
        row("a6 scaled LayerNorm bwd + exact dynamic L2 rescale to E5M2 in ONE pass (dX = NULL: rebalanced with the "
            "predicted power of two, repair launch returns at once when it held; 5 B/elem + 8 B/row; bit-identical to "
            "the two-pass row below, checked)", seg_ms[5], 5 * n_ln + 8 * LN_R),
        row("a6 as two passes with the BF16 intermediate stored (second pass of the same step, 9 B/elem + 8 B/row)",
            ln_two_pass_ms, 9 * n_ln + 8 * LN_R),
        row("a7 scaled Adam, E5M2 grads, FP16 m/v/w (13 B/param)", seg_ms[6], 13 * ADAM_N),
        {"row": "f1 (next, timed outside the step, back to back) delayed-rescale GEMM 8192^3: E4M3 out in one "
                "kernel, no BF16 intermediate, no pass 2", "ms": round(float(delayed_ms), 4),
         "TFLOP/s": round(flops / (delayed_ms * 1e-3) / 1e12, 1)},
        row("f1 (next, timed outside the step, back to back) LayerNorm bwd with delayed L2 rescale: E5M2 gradient "
            "in one pass, no BF16 intermediate, no pass 2 (5 B/elem + 8 B/row)", ln_delayed_ms, 5 * n_ln + 8 * LN_R),
        {"row": "f1b (next, timed in a third pass of the same step) the headline call with Y = NULL: only the E4M3 "
                "output is stored (values still rounded through BF16, AMAX of the BF16 values; a repair launch of the "
                "same kernel returns at once when the prediction held); Yq, scale and statistic bit-identical",
         "ms": round(float(fp8_only_ms), 4), "TFLOP/s": round(flops / (fp8_only_ms * 1e-3) / 1e12, 1)},
        row("f2 (next, timed outside the step, back to back) scaled Adam that also writes the E4M3 compute copy "
            "of the weight (14 B/param)", adam_cast_ms, 14 * ADAM_N),
        row("f3 (next, own loop) block-scale quantisation of two 8192^2 BF16 operands to E4M3 + E8M0 per 32 "
            "elements (3.03 B/elem)", mx_q_ms, 2 * (3 * N_GEMM * N_GEMM + N_GEMM * N_GEMM // 32)),
        {"row": "f3 (next, own loop) block-scaled GEMM 8192^3 (tcgen05 kind::mxf8f6f4.block_scale, two-CTA tiles), "
                "BF16 out + fused AMAX", "ms": round(float(mx_mm_ms), 4),
         "TFLOP/s": round(flops / (mx_mm_ms * 1e-3) / 1e12, 1)},
        row("f3 (next, own loop) block-scale quantisation, transposed form: operands stored [K, rows], blocks of 32 "
            "down the columns (3.03 B/elem)", mx_qt_ms, 2 * (3 * N_GEMM * N_GEMM + N_GEMM * N_GEMM // 32)),
        {"row": "f3 (next, own loop) block-scaled GEMM 8192^3, both operands in the transposed (MN-major) form of "
                "the gradient products", "ms": round(float(mx_mmt_ms), 4),
         "TFLOP/s": round(flops / (mx_mmt_ms * 1e-3) / 1e12, 1)},
        {"row": f"f4 (next, own loop over {ATT_SETS} buffer sets) fused causal attention forward, 96 heads x 1024 tokens "
                "x 64 (scores and probabilities never leave the chip)", "ms": round(float(att_ms), 4),
         "TFLOP/s": round(2.0 * ATT_H * ATT_T * ATT_T * ATT_HD / (att_ms * 1e-3) / 1e12, 1),
         "ms_cuda_graph": round(float(att_graph_ms), 4),
         "note": "flop counted for the causal half of Q K^T and P V; ms_cuda_graph: the same calls replayed from a "
                 "CUDA graph (the call from Python takes longer than the kernel runs)"},
        {"row": "f4 (next, own loop) fused causal attention backward, same shape: dQ, dK, dV from dO and the "
                "forward's E4M3 probabilities in two launches (dP never leaves the chip, dS is written once)",
         "ms": round(float(att_bwd_ms), 4),
         "TFLOP/s": round(4.0 * ATT_H * ATT_T * ATT_T * ATT_HD / (att_bwd_ms * 1e-3) / 1e12, 1),
         "ms_cuda_graph": round(float(att_bwd_graph_ms), 4),
         "note": "flop counted for the causal half of dO V^T, dS K, dS^T Q and P^T dO; ms_cuda_graph as above"},
    ] + sweep_rows
    # Which of the two measured bf16 rates is the denominator: the sustained one holds for a GEMM that runs for
    # seconds under the power cap; a timed region under a second, or a GEMM that is less than half of the step's
    # duty cycle, runs at burst clocks.
    gemm_share = float(seg_ms[0]) / float(np.sum(seg_ms))
    burst = total_ms < 1000.0 or gemm_share < 0.5
    # the dominant kernel's duration over the timed region: the headline call is that kernel plus a check launch
    # of a few microseconds, so this is an upper bound on the kernel's own time (its own time, from the second
    # pass of the step, is reported beside it)
    gemm_tflops = flops / (float(seg_ms[0]) * 1e-3) / 1e12
    gemm_alone_tflops = flops / (two_call_ms[0] * 1e-3) / 1e12
    peak_burst, peak_sust = 2.0 * peaks["bf16_burst"], 2.0 * peaks["bf16_sustained"]
    fp8_peak = peak_burst if burst else peak_sust
    roofline = {
        "bound": "tensor", "kernel": "scaled_matmul_spec_kernel<BF16> (tcgen05 kind::f8f6f4; BF16 + E4M3 outputs, fused AMAX)",
        "achieved": round(gemm_tflops, 1), "peak": round(fp8_peak, 1), "unit": "TFLOP/s",
        "frac": round(gemm_tflops / fp8_peak, 4),
        "frac_vs_burst": round(gemm_tflops / peak_burst, 4), "frac_vs_sustained": round(gemm_tflops / peak_sust, 4),
        "achieved_note": "flop / duration of the headline call (kernel + check launch) over the timed region",
        "achieved_plain_gemm_alone": round(gemm_alone_tflops, 1),
        "peak_source": f"{peaks['source']}: 2 x {'burst' if burst else 'sustained'} bf16 cuBLAS "
                       f"({peaks['bf16_burst'] if burst else peaks['bf16_sustained']} TFLOP/s), fp8:bf16 nominal ratio 2 "
                       f"(timed region {total_ms:.0f} ms, GEMM {100 * gemm_share:.0f} % of it); nominal dense fp8 4500",
        "frac_of_nominal_4500": round(gemm_tflops / 4500.0, 4),
        "traffic": gemm_dram_traffic(),
    }
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp8 (e4m3 x e4m3, fp32 accumulate)", "data": "synthetic",
        "config": {"workload": f"configs[1]: scaled GEMM M=N=K={N_GEMM} forward E4M3xE4M3, BF16 intermediate + fused "
                               "AMAX + rescale to E4M3 in one call; the step also runs the two-call form and rows "
                               "a3'-a7, and the other sizes and the gradient formats of configs[1] follow in rows",
                   "l2": "inputs larger than L2: every step streams > 5 GB, so no operand survives in L2 between "
                         "iterations", "replicas": world},
        "headline_ms": round(head_ms_max, 4),
        "rows": rows,
        "roofline": roofline,
        "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "ms": round(e2e_ms_max, 3),
                "h2d_bytes_per_step": int(hA.numel() + hB.numel()), "d2h_bytes_per_step": int(hY.numel() + 4),
                "pipeline": "copy-in, kernels and copy-out of consecutive steps overlap on three streams "
                            "(two buffer sets); every step copies its own inputs and result"},
        "gpu_launches": launches_per_step * K,
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        import oracle as orc
        v, dt = oracle_sample(ORACLE_SAMPLE_ROWS)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                                "sample": f"{ORACLE_SAMPLE_ROWS} of {N_GEMM} output rows of the 8192^3 GEMM + AMAX "
                                          f"rescale of those rows ({dt:.1f} s)"}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
