"""Benchmark of the ARL^2 hybrid attention layer on B200.

A bench "step" is one autoregressive block of the layer's whole hot path: `n_steps` denoise
passes (intra-block softmax + state readout + gated combine, the state only read) followed by
one state commit.  The metric is tokens per second through the denoise passes, with the commit
time included:  value = N_gpus * B * L * n_steps / t_block.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload long] [--impl reference]

N > 1 is launched by torchrun, one rank per GPU.  The layer shards by (stream, head) with no
exchange inside it, so ranks are independent replicas ("weak" scaling); torch.distributed is
used only for the barrier and the max-over-ranks of the device time.

`--impl reference` times the CPU float64 checker (as it stands) on the host cores, on bounded
samples of the same workload, and prints the same JSON line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "hybrid-attn layer tokens/s per denoise step"
UNIT = "tokens/s"
RING = 3  # pre-generated step-input sets the timed loop rotates through
HORIZON_BLOCKS = 120  # blocks of the timed loop whose individual latency is recorded (config 5's horizon)


def peaks():
    """Measured roofline denominators of this machine's B200s, else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def workload_text(cfg):
    return (f"{cfg.name}: B={cfg.B} H={cfg.H} D={cfg.D} L={cfg.L} {cfg.dtype}, "
            f"{cfg.steps} denoise steps + 1 commit per block")


def step_flops(cfg):
    """Algorithmic tensor flops of one denoise pass: QK^T, PV, Q W_phi_q, Q' S."""
    return cfg.B * cfg.H * (4.0 * cfg.L * cfg.L * cfg.D + 4.0 * cfg.L * cfg.D * cfg.D)


def commit_bytes_flops(cfg):
    """Algorithmic HBM bytes and tensor flops of one gated-linear commit: K_c, V_c in, S read and
    written, the two maps; U_k, U_v and K'^T V' contractions."""
    e = cfg.elem_bytes
    byts = cfg.B * cfg.H * (2.0 * cfg.L * cfg.D * e + 8.0 * cfg.D * cfg.D + 2.0 * cfg.D * cfg.D * e)
    flops = cfg.B * cfg.H * 6.0 * cfg.L * cfg.D * cfg.D
    return byts, flops


def step_bytes(cfg):
    """Algorithmic HBM bytes of one denoise pass: Q, K, V in, O out, gate logits, S and W_phi_q."""
    e = cfg.elem_bytes
    return cfg.B * cfg.H * (4.0 * cfg.L * cfg.D * e + 4.0 * cfg.L + cfg.D * cfg.D * (4 + e))


def sfu_bound(cfg, kern_ms, sm_mhz, per_clk_per_sm=16, sms=148):
    """Exponentials of one denoise pass against the special-function unit's rate."""
    n_exp = float(cfg.B * cfg.H) * cfg.L * cfg.L
    if not sm_mhz:
        return {"exp_per_launch": n_exp, "min_ms": None, "frac": None}
    min_ms = n_exp / (per_clk_per_sm * sms * sm_mhz * 1e6) * 1e3
    return {"exp_per_launch": n_exp, "min_ms": min_ms, "frac": min_ms / kern_ms,
            "rate": f"{per_clk_per_sm}/clk/SM x {sms} SMs at {sm_mhz:.0f} MHz"}


class ClockSampler:
    """nvidia-smi in the background during the timed region (read-only queries)."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc, self.index = None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for n, val in zip(names, parts[3:7]):
                if val.lower() == "active":
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm),
                "power_w_max": max(power), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------
# CPU checker timings (the "reference arm" of this tier and the cpu_baseline leg)
# ------------------------------------------------------------------------------------------

class CpuSample:
    """Times the CPU float64 checker on a bounded sample of one block of `cfg`."""

    def __init__(self, cfg):
        import numpy as np

        from oracle import arl2_oracle
        from paper_2605_16579_b200 import workload

        self.np, self.o, self.cfg = np, arl2_oracle, cfg
        self.threads = arl2_oracle.threads()
        f64 = lambda t: None if t is None else t.double().numpy()  # noqa: E731
        q, k, v, g = workload.step_inputs(cfg, 0, 0)
        kc, vc, a = workload.commit_inputs(cfg, 0)
        self.q, self.k, self.v, self.g = f64(q), f64(k), f64(v), f64(g)
        self.kc, self.vc, self.a = f64(kc), f64(vc), f64(a)
        wq, wk, wv = workload.feature_weights(cfg)
        cos, sin = workload.rope_tables(cfg.L, cfg.D)
        self.wq, self.wk, self.wv, self.cos, self.sin = f64(wq), f64(wk), f64(wv), f64(cos), f64(sin)
        rng = np.random.default_rng(1)
        self.S = rng.standard_normal((cfg.B, cfg.H, cfg.D, cfg.D)) * 0.1
        self.rng = rng

    def time_rows(self, n):
        cfg, np = self.cfg, self.np
        rows = np.stack([self.rng.integers(0, cfg.B, n), self.rng.integers(0, cfg.H, n),
                         self.rng.integers(0, cfg.L, n)], axis=1)
        t0 = time.perf_counter()
        self.o.step_rows(self.q, self.k, self.v, self.g, self.S, rows, self.wq, self.cos, self.sin)
        return time.perf_counter() - t0

    def time_heads(self, n):
        cfg = self.cfg
        heads = [((i // cfg.H) % cfg.B, i % cfg.H) for i in range(n)]
        t0 = time.perf_counter()
        self.o.commit(self.kc, self.vc, self.a, self.S, self.wk, self.wv, self.cos, self.sin,
                      heads=heads)
        return time.perf_counter() - t0

    def block_seconds(self, n_rows, t_rows, n_heads, t_heads):
        """Extrapolate one block (n_steps denoise passes + commit) from the sample rates."""
        cfg = self.cfg
        rows_per_step = cfg.B * cfg.L * cfg.H
        return cfg.steps * rows_per_step * (t_rows / n_rows) + cfg.B * cfg.H * (t_heads / n_heads)


def run_reference(args):
    from paper_2605_16579_b200 import workload

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = workload.CONFIGS[args.workload]
    s = CpuSample(cfg)
    target = min(1.0, 150.0 / max(args.steps + args.warmup, 1))  # seconds of CPU work per step
    t = s.time_rows(s.threads)  # calibration
    n_rows = max(s.threads, int(s.threads * (0.8 * target) / max(t, 1e-6)))
    n_heads = 1 if s.time_heads(1) > 0.2 * target else min(s.threads, cfg.B * cfg.H)
    for _ in range(args.warmup):
        s.time_rows(n_rows)
    per_step, est = [], []
    for _ in range(args.steps):
        tr = s.time_rows(n_rows)
        th = s.time_heads(n_heads)
        per_step.append(tr + th)
        est.append(s.block_seconds(n_rows, tr, n_heads, th))
    block_s = statistics.mean(est)
    value = cfg.B * cfg.L * cfg.steps / block_s
    sample = (f"per step: {n_rows} random output rows (b,h,i) of one denoise pass + commit of "
              f"{n_heads} head(s), extrapolated to {cfg.steps} passes over B*L*H = "
              f"{cfg.B * cfg.L * cfg.H} rows and {cfg.B * cfg.H} heads")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * statistics.mean(per_step), "extrapolated_block_ms": 1e3 * block_s,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": workload_text(cfg)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": s.threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------

def max_over_ranks(values, world, device):
    """Device times of the replicas -> the slowest rank's (all ranks get the same list)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist

    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def horizon_report(block_ms, mem_marks, layer_bytes):
    """Per-block latency and device memory against the number of past blocks: the layer keeps a
    fixed-size state per (stream, head), so both must stay flat however long the video gets."""
    n = len(block_ms)
    if n < 4:
        return None
    q = max(n // 10, 1)
    return {
        "blocks": n,
        "ms_first": statistics.mean(block_ms[:q]), "ms_last": statistics.mean(block_ms[-q:]),
        "ms_min": min(block_ms), "ms_max": max(block_ms),
        "last_over_first": statistics.mean(block_ms[-q:]) / statistics.mean(block_ms[:q]),
        # the first blocks run before the power cap pulls the SM clock down; the middle and last
        # thirds run at the settled clock and isolate the dependence on the horizon itself
        "ms_mid_third": statistics.mean(block_ms[n // 3:2 * n // 3]),
        "ms_last_third": statistics.mean(block_ms[2 * n // 3:]),
        "last_third_over_mid_third": statistics.mean(block_ms[2 * n // 3:]) / statistics.mean(block_ms[n // 3:2 * n // 3]),
        "device_bytes_first": mem_marks[0], "device_bytes_last": mem_marks[-1],
        "state_plus_workspace_bytes": layer_bytes,
    }


def rank_seeds(rank):
    """Each replica draws its own inputs: step-input seeds and the commit block index."""
    return [s + 10 * rank for s in range(RING)], rank


def whole_job_value(cfg, world, ms_block):
    """tokens/s through the denoise passes of all replicas, commit time included."""
    return world * cfg.B * cfg.L * cfg.steps / (ms_block * 1e-3)


def step_traffic(cfg, kernel_name):
    """DRAM bytes of one launch of the step kernel from the committed profiler capture: the figure
    captured at this very shape when there is one, else a smaller capture scaled by the number of
    (stream, head) units (heads share only the rotation table), else None."""
    tpath = os.path.join(ROOT, "profiles", "step_kernel_traffic.txt")
    if not os.path.exists(tpath):
        return None, "no capture committed"
    with open(tpath) as f:
        recs = json.load(f)
    recs = recs if isinstance(recs, list) else [recs]
    recs = [r for r in recs if r.get("step_kernel") == kernel_name]
    for r in recs:
        if r.get("shape") == [cfg.B, cfg.H, cfg.L, cfg.D]:
            return r["dram_bytes_per_launch"], "captured at this shape: " + r["source"]
    for r in recs:
        if r.get("shape", [0, 0, cfg.L, cfg.D])[2:] == [cfg.L, cfg.D]:
            return (r["dram_bytes_per_head"] * cfg.B * cfg.H,
                    f"scaled by (stream, head) count from {r['captured_workload']}: " + r["source"])
    return None, "no capture of this per-head shape"


def short_leg(name, dev, blocks=8):
    """A short run of another workload beside the main one: tokens/s per block and the step kernel's
    rate.  Three warm-up blocks, then `blocks` timed ones; inputs rotate through resident sets that
    together exceed the L2 cache (two at least)."""
    import torch

    from paper_2605_16579_b200 import arl2, workload

    cfg = workload.CONFIGS[name]
    pk = peaks()
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=dev)
    wq, wk, wv = (w.to(dev) for w in workload.feature_weights(cfg))
    cos, sin = (t.to(dev) for t in workload.rope_tables(cfg.L, cfg.D))
    layer.set_params(wq, wk, wv, cos, sin)
    set_bytes = (3 * cfg.D * 2 + 4) * cfg.B * cfg.L * cfg.H
    nsets = max(2, -(-(160 << 20) // set_bytes))
    sets = [tuple(t.to(dev) for t in workload.step_inputs(cfg, 0, s)) for s in range(nsets)]
    kc, vc, a = (t.to(dev) for t in workload.commit_inputs(cfg, 0))
    out = torch.empty(cfg.B, cfg.L, cfg.H, cfg.D, dtype=cfg.torch_dtype, device=dev)
    events = []
    calls = [0]

    def block(timed):
        for s in range(cfg.steps):
            if timed:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                layer.set_profile_events(e0, e1)
                events.append((e0, e1))
            layer.denoise_step(*sets[calls[0] % nsets], out=out)
            calls[0] += 1
        layer.commit(kc, vc, a)

    for _ in range(3):
        block(False)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(blocks):
        block(True)
    t1.record()
    torch.cuda.synchronize()
    layer.sync_status()
    ms_block = t0.elapsed_time(t1) / blocks
    kern = statistics.mean(a_.elapsed_time(b_) for a_, b_ in events)
    tf = step_flops(cfg) / (kern * 1e-3) / 1e12
    return {"workload": workload_text(cfg), "blocks_timed": blocks, "ms_per_block": ms_block,
            "tokens_per_s": cfg.B * cfg.L * cfg.steps / (ms_block * 1e-3), "step_kernel_ms": kern,
            "step_kernel_tflops": tf, "frac_of_burst": tf / pk["bf16_tflops"],
            "frac_of_sustained": tf / pk["bf16_tflops_sustained"],
            "l2": "%d resident input sets of %d MiB" % (nsets, sum(t.numel() * t.element_size() for t in sets[0]) >> 20)}


def stack_leg(dev, horizons=(1, 2, 4, 8, 16), n_layers=30, n_hybrid=23):
    """The attention modules of a whole model, measured: 30 layers of (x -> W_q | W_k | W_v | W_g -> attention
    core -> W_o) per denoise pass at the base model's geometry (d = 1536, H = 12, 4680 tokens per block), once
    with every layer a softmax teacher over a key/value cache of n blocks (Eq. 1) and once with 23 of the 30
    layers replaced by the hybrid layer (the paper's 75 % model).  Every layer has its own weights, state and
    cache; the feed-forward blocks, norms and residuals between the attention modules are not part of this
    path and are left out of both arms.  Returns ms per pass against the horizon and the GEMM rates."""
    import torch

    from paper_2605_16579_b200 import arl2, workload

    cfg = workload.CONFIGS["chunked"]
    pk = peaks()
    B, H, L, D = cfg.B, cfg.H, cfg.L, cfg.D
    d = H * D
    gen = torch.Generator(device="cpu").manual_seed(4242)
    rnd = lambda *s: (torch.randn(*s, generator=gen) * d ** -0.5).to(torch.bfloat16).to(dev)  # noqa: E731
    wq, wk, wv = (w.to(dev) for w in workload.feature_weights(cfg))
    cos, sin = (t.to(dev) for t in workload.rope_tables(L, D))
    layers = []
    for _ in range(n_layers):
        layer = arl2.Layer(B, H, L, D, "bf16", device=dev)
        layer.set_params(wq, wk, wv, cos, sin)
        layer.set_projections(rnd(d, d), rnd(d, d), rnd(d, d), rnd(d, H), rnd(d, d))
        kc, vc, a = (t.to(dev) for t in workload.commit_inputs(cfg, 0))
        layer.commit(kc, vc, a)
        layers.append(layer)
    nmax = max(horizons)
    caches = [(torch.randn(B, nmax * L, H, D, device=dev).to(torch.bfloat16),
               torch.randn(B, nmax * L, H, D, device=dev).to(torch.bfloat16)) for _ in range(n_layers)]
    xs = [torch.randn(B, L, d, device=dev).to(torch.bfloat16) for _ in range(2)]
    q = torch.empty(B, L, H, D, dtype=torch.bfloat16, device=dev)
    k, v, o = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    g = torch.empty(B, L, H, device=dev)

    def one_pass(hybrid_set, n):
        x, y = xs
        for i, layer in enumerate(layers):
            if i in hybrid_set:
                layer.project_in(x, q, k, v, g)
                layer.denoise_step(q, k, v, g, out=o)
            else:
                # the block's keys and values land at the tail of this layer's cache
                ck, cv = caches[i]
                k_cur, v_cur = ck[:, (n - 1) * L:n * L], cv[:, (n - 1) * L:n * L]
                layer.project_in(x, q, k_cur, v_cur, g)
                layer.teacher_step(q, ck[:, :n * L], cv[:, :n * L], out=o)
            layer.project_out(o, y)
            x, y = y, x

    def timed(hybrid_set, n, reps=4):
        for _ in range(2):
            one_pass(hybrid_set, n)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            one_pass(hybrid_set, n)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    # which layers stay softmax: spread over the depth (the paper selects them by sensitivity; the cost
    # does not depend on which ones they are)
    keep = {round(j * (n_layers - 1) / (n_layers - n_hybrid - 1)) for j in range(n_layers - n_hybrid)}
    hybrid_set = set(range(n_layers)) - keep
    res = {"geometry": f"B={B} H={H} D={D} d={d} L={L}, {n_layers} layers, {n_hybrid} hybrid + {n_layers - n_hybrid} softmax",
           "cache_blocks": list(horizons), "all_softmax_ms": [], "hybrid75_ms": [], "speedup": []}
    for n in horizons:
        t_all = timed(set(), n)
        t_hyb = timed(hybrid_set, n)
        res["all_softmax_ms"].append(t_all)
        res["hybrid75_ms"].append(t_hyb)
        res["speedup"].append(t_all / t_hyb)
    # the two GEMMs on their own
    def gemm_ms(fn, reps=20):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps
    t_in = gemm_ms(lambda i=0: layers[i % n_layers].project_in(xs[0], q, k, v, g))
    t_out = gemm_ms(lambda i=0: layers[i % n_layers].project_out(o, xs[1]))
    f_in, f_out = 2.0 * B * L * d * (3 * d + H), 2.0 * B * L * d * d
    res["project_in"] = {"ms": t_in, "tflops": f_in / t_in / 1e9, "frac_of_burst": f_in / t_in / 1e9 / pk["bf16_tflops"]}
    res["project_out"] = {"ms": t_out, "tflops": f_out / t_out / 1e9, "frac_of_burst": f_out / t_out / 1e9 / pk["bf16_tflops"]}
    res["kv_cache_bytes_per_block_per_layer"] = 2 * B * L * d * 2
    res["state_bytes_per_layer"] = B * H * D * D * 4
    for layer in layers:
        layer.sync_status()
    return res


def launcher_command(n, argv, port=None):
    """The command that runs this file as n ranks of one node (what a caller would type)."""
    port = port or 29400 + os.getpid() % 500
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def run_traffic_probe(args):
    """A minimal run for a profiler: the layer is set up, three denoise passes warm up, one more
    runs, the process ends.  Used to read the DRAM bytes of ONE launch of the dominant kernel at
    the bench's own shape (two counters of one hardware unit: a single replay pass)."""
    import torch

    from paper_2605_16579_b200 import arl2, workload

    arl2.load(build_if_missing=True)
    dev = torch.device("cuda", 0)
    cfg = workload.CONFIGS[args.workload]
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=dev)
    wq, wk, wv = (w.to(dev) for w in workload.feature_weights(cfg))
    cos, sin = (t.to(dev) for t in workload.rope_tables(cfg.L, cfg.D))
    layer.set_params(wq, wk, wv, cos, sin)
    sets = [tuple(t.to(dev) for t in workload.step_inputs(cfg, 0, s)) for s in range(RING)]
    kc, vc, a = (t.to(dev) for t in workload.commit_inputs(cfg, 0))
    layer.commit(kc, vc, a)
    out = torch.empty(cfg.B, cfg.L, cfg.H, cfg.D, dtype=cfg.torch_dtype, device=dev)
    for i in range(4):
        layer.denoise_step(*sets[i % RING], out=out)
    layer.commit(kc, vc, a)
    if args.probe_all and cfg.dtype == "bf16" and cfg.D == 128:
        # one call of every other entry point, so that one small command shows every kernel
        q, k, v, g = sets[0]
        layer.clean_pass(q, kc, vc, g, a, out=out)
        layer.commit_delta(kc, vc, a, workload.beta_logits(cfg, 0).to(dev))
        alpha, _ = (t.to(dev) for t in workload.token_gate_logits(cfg, 0))
        layer.commit_decay_tokens(kc, vc, alpha)
        layer.denoise_step_token_level(q, k, v, g, alpha, out=out)
        d = cfg.H * cfg.D
        gen = torch.Generator(device="cpu").manual_seed(4242)
        rnd = lambda *s: (torch.randn(*s, generator=gen) * d ** -0.5).to(torch.bfloat16).to(dev)  # noqa: E731
        layer.set_projections(rnd(d, d), rnd(d, d), rnd(d, d), rnd(d, cfg.H), rnd(d, d))
        x = torch.randn(cfg.B, cfg.L, d, generator=gen).to(torch.bfloat16).to(dev)
        pq, pk_, pv, pg = layer.project_in(x)
        layer.project_out(pq)
    layer.sync_status()
    print(json.dumps({"traffic_probe": workload_text(cfg), "launches": layer.launch_count}))


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2605_16579_b200 import arl2, workload

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    arl2.load(build_if_missing=True)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    cfg = workload.CONFIGS[args.workload]
    layer = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=dev)
    wq, wk, wv = (w.to(dev) for w in workload.feature_weights(cfg))
    cos, sin = (t.to(dev) for t in workload.rope_tables(cfg.L, cfg.D))
    layer.set_params(wq, wk, wv, cos, sin)

    step_seeds, commit_block = rank_seeds(rank)
    host_sets = [workload.step_inputs(cfg, 0, s) for s in step_seeds]
    host_commit = workload.commit_inputs(cfg, commit_block)
    dev_sets = [tuple(t.to(dev) for t in hs) for hs in host_sets]
    dev_commit = tuple(t.to(dev) for t in host_commit)
    out = torch.empty(cfg.B, cfg.L, cfg.H, cfg.D, dtype=cfg.torch_dtype, device=dev)
    set_bytes = sum(t.numel() * t.element_size() for t in host_sets[0])

    step_events = []
    pass_events = []   # around the whole call: the K rotation launch and the fused kernel

    def block(i, timed):
        for s in range(cfg.steps):
            q, k, v, g = dev_sets[(i * cfg.steps + s) % RING]
            if timed:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                layer.set_profile_events(e0, e1)
                step_events.append((e0, e1))
                p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                pass_events.append((p0, p1))
                p0.record()
            layer.denoise_step(q, k, v, g, out=out)
            if timed:
                p1.record()
        layer.commit(*dev_commit)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        block(i, False)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = layer.launch_count
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    block_marks = [t0]      # one event per block boundary: per-block latency against the horizon
    mem_marks = []
    for i in range(args.steps):
        block(i, True)
        if i < HORIZON_BLOCKS:
            ev = torch.cuda.Event(enable_timing=True)
            ev.record()
            block_marks.append(ev)
            mem_marks.append(torch.cuda.memory_allocated(dev))
    t1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    launches = layer.launch_count - launches0
    ms_total = t0.elapsed_time(t1)
    kern_ms = [a.elapsed_time(b) for a, b in step_events]
    pass_ms = [a.elapsed_time(b) for a, b in pass_events]
    block_ms = [block_marks[i].elapsed_time(block_marks[i + 1]) for i in range(len(block_marks) - 1)]
    layer.sync_status()

    # end to end through the same entry points with HOST buffers: every pass copies its inputs
    # from pinned host memory and its output back inside the timed region.  Copies run on their own
    # streams with double-buffered staging, as a caller would: the upload of the next pass and the
    # download of the previous one overlap the kernels (PCIe carries both directions at once).
    e2e_blocks = max(1, min(args.steps, 5))
    pin_sets = [tuple(t.pin_memory() for t in hs) for hs in host_sets]
    pin_commit = tuple(t.pin_memory() for t in host_commit)
    pin_outs = [torch.empty(out.shape, dtype=out.dtype).pin_memory() for _ in range(2)]
    stages = [tuple(torch.empty_like(t) for t in dev_sets[0]) for _ in range(2)]
    outs = [torch.empty_like(out) for _ in range(2)]
    stage_c = tuple(torch.empty_like(t) for t in dev_commit)
    s_main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]        # staging slot filled
    ev_done = [torch.cuda.Event() for _ in range(2)]      # kernels of the slot finished
    ev_out = [torch.cuda.Event() for _ in range(2)]       # output slot downloaded
    ev_c_in, ev_c_done = torch.cuda.Event(), torch.cuda.Event()
    for e in ev_done + ev_out + [ev_c_done]:
        e.record(s_main)
    n_pass = [0]

    def block_host(i):
        for s in range(cfg.steps):
            slot = n_pass[0] & 1
            n_pass[0] += 1
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_done[slot])            # the kernels that read this slot are done
                for d, h in zip(stages[slot], pin_sets[(i * cfg.steps + s) % RING]):
                    d.copy_(h, non_blocking=True)
                ev_in[slot].record(s_in)
            s_main.wait_event(ev_in[slot])
            s_main.wait_event(ev_out[slot])               # the previous output of this slot is on the host
            layer.denoise_step(*stages[slot], out=outs[slot])
            ev_done[slot].record(s_main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[slot])
                pin_outs[slot].copy_(outs[slot], non_blocking=True)
                ev_out[slot].record(s_out)
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_c_done)
            for d, h in zip(stage_c, pin_commit):
                d.copy_(h, non_blocking=True)
            ev_c_in.record(s_in)
        s_main.wait_event(ev_c_in)
        layer.commit(*stage_c)
        ev_c_done.record(s_main)

    def drain():
        s_main.wait_stream(s_in)
        s_main.wait_stream(s_out)

    block_host(0)
    drain()
    barrier()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record()
    for i in range(e2e_blocks):
        block_host(i)
    drain()                                               # every download has landed before the clock stops
    h1.record()
    barrier()
    ms_e2e = h0.elapsed_time(h1)
    commit_bytes = sum(t.numel() * t.element_size() for t in host_commit)
    h2d = cfg.steps * set_bytes + commit_bytes
    d2h = cfg.steps * out.numel() * out.element_size()

    # the two commit rules side by side (outside the timed regions above): the gated-linear commit
    # the block uses, and the delta rule of Eq. 4 at block level
    beta = workload.beta_logits(cfg, commit_block).to(dev)
    commit_ms = {}
    alpha_tok = workload.token_gate_logits(cfg, commit_block)[0].to(dev)
    for name, call in (("gated_linear", lambda: layer.commit(*dev_commit)),
                       ("delta", lambda: layer.commit_delta(*dev_commit, beta)),
                       ("decay_tokens", lambda: layer.commit_decay_tokens(dev_commit[0], dev_commit[1], alpha_tok))):
        layer.reset()
        for _ in range(3):
            call()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for _ in range(20):
            call()
        c1.record()
        torch.cuda.synchronize()
        commit_ms[name] = c0.elapsed_time(c1) / 20
    layer.sync_status()
    # Eq. 4 token by token with per-token gates: needs a context with the extra workspace
    tok = arl2.Layer(cfg.B, cfg.H, cfg.L, cfg.D, cfg.dtype, device=dev, flags=arl2.ARL2_FLAG_TOKEN_GATES)
    tok.set_params(wq, wk, wv, cos, sin)
    tok.reset()
    gates = tuple(t.to(dev) for t in workload.token_gate_logits(cfg, commit_block))
    for _ in range(2):
        tok.commit_tokens(dev_commit[0], dev_commit[1], *gates)
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record()
    for _ in range(10):
        tok.commit_tokens(dev_commit[0], dev_commit[1], *gates)
    c1.record()
    torch.cuda.synchronize()
    commit_ms["token_gates"] = c0.elapsed_time(c1) / 10
    tok.sync_status()
    del tok

    # the clean pass of a block: the fused call against the two separate calls, alternating so that
    # both see the same clocks; and the token-level state access mode beside the frame-level pass
    clean_ms = None
    if layer.step_kernel == "tcgen05":
        q0, _, _, g0 = dev_sets[0]
        kc0, vc0, a0 = dev_commit

        def run_ms(fn, reps):
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            for _ in range(reps):
                fn()
            c1.record()
            torch.cuda.synchronize()
            return c0.elapsed_time(c1) / reps

        def two_calls():
            layer.denoise_step(q0, kc0, vc0, g0, out=out)
            layer.commit(kc0, vc0, a0)

        def fused():
            layer.clean_pass(q0, kc0, vc0, g0, a0, out=out)

        layer.reset()
        for fn in (two_calls, fused):
            run_ms(fn, 3)
        t_two, t_fused = [], []
        for _ in range(4):
            t_two.append(run_ms(two_calls, 8))
            t_fused.append(run_ms(fused, 8))
        alpha0 = workload.token_gate_logits(cfg, commit_block)[0].to(dev)
        run_ms(lambda: layer.denoise_step_token_level(q0, kc0, vc0, g0, alpha0, out=out), 2)
        t_tok = run_ms(lambda: layer.denoise_step_token_level(q0, kc0, vc0, g0, alpha0, out=out), 5)
        t_frame = run_ms(lambda: layer.denoise_step(q0, kc0, vc0, g0, out=out), 5)
        clean_ms = {"step_then_commit": statistics.median(t_two), "clean_pass": statistics.median(t_fused),
                    "frame_level_pass": t_frame, "token_level_pass": t_tok}
        layer.sync_status()
        layer.reset()

    # the teacher's layer on the same kernels (Eq. 1 over a key/value cache that grows by one block
    # per generated block) against the horizon: its cost per denoise pass grows, the layer's does not
    teacher = None
    if layer.step_kernel == "tcgen05" and not args.no_teacher:
        teacher = {"cache_blocks": [], "ms_per_pass": []}
        q0, k0, v0, _ = dev_sets[0]
        for nb in (1, 2, 4, 8, 16):
            kcache, vcache = k0.repeat(1, nb, 1, 1), v0.repeat(1, nb, 1, 1)
            ts = []
            for it in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                layer.set_profile_events(e0, e1)
                layer.teacher_step(q0, kcache, vcache, out=out)
                torch.cuda.synchronize()
                if it >= 2:
                    ts.append(e0.elapsed_time(e1))
            teacher["cache_blocks"].append(nb)
            teacher["ms_per_pass"].append(statistics.mean(ts))
            del kcache, vcache
        layer.sync_status()
    batched, chunked = None, None
    if rank == 0 and world == 1 and cfg.name == "long" and not args.no_batched_leg:
        batched = short_leg("batched", dev, blocks=8)
        chunked = short_leg("chunked", dev, blocks=16)
    stack = None
    if rank == 0 and world == 1 and layer.step_kernel == "tcgen05" and not args.no_stack:
        stack = stack_leg(dev)

    ms_total, ms_e2e, kern_mean, pass_mean = max_over_ranks(
        [ms_total, ms_e2e, statistics.mean(kern_ms), statistics.mean(pass_ms)], world, dev)

    if rank == 0:
        pk = peaks()
        ms_block = ms_total / args.steps
        value = whole_job_value(cfg, world, ms_block)
        # the denominator is always the burst figure (cuBLAS bf16 timed alone): the stricter of the
        # two measured peaks, and the same whatever the run length; the fraction of the sustained
        # figure (a seconds-long loop under the power cap, which is how this kernel is timed at the
        # default run length) is printed beside it
        peak = pk["bf16_tflops"]
        achieved = step_flops(cfg) / (kern_mean * 1e-3) / 1e12
        traffic, traffic_note = step_traffic(cfg, layer.step_kernel)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_block, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {
                "workload": workload_text(cfg),
                "step_definition": "one AR block = n_steps denoise passes + 1 state commit",
                "l2": f"inputs larger than L2: ring of {RING} input sets of {set_bytes >> 20} MiB",
                "parallelism": "replicas" if world > 1 else "single GPU",
                "step_kernel": layer.step_kernel,
            },
            "denoise_pass": {"kernel_ms_mean": kern_mean, "kernel_ms_median": statistics.median(kern_ms),
                             "tokens_per_s": cfg.B * cfg.L / (kern_mean * 1e-3)},
            # the whole arl2_denoise_step call: the K rotation launch and the fused kernel
            "denoise_pass_all_kernels": {
                "ms_mean": pass_mean, "tflops": step_flops(cfg) / (pass_mean * 1e-3) / 1e12,
                "frac_of_burst": step_flops(cfg) / (pass_mean * 1e-3) / 1e12 / pk["bf16_tflops"],
                "frac_of_sustained": step_flops(cfg) / (pass_mean * 1e-3) / 1e12 / pk["bf16_tflops_sustained"]},
            # the whole block (denoise passes + commit), i.e. `value` as a fraction of the tensor peak
            "block_all_kernels": {
                "frac_of_burst": cfg.steps * step_flops(cfg) / (ms_block * 1e-3) / 1e12 / pk["bf16_tflops"],
                "frac_of_sustained": cfg.steps * step_flops(cfg) / (ms_block * 1e-3) / 1e12 / pk["bf16_tflops_sustained"]},
            "roofline": {
                "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": traffic, "traffic_note": traffic_note,
                "peak_kind": "burst bf16, " + pk["source"],
                "frac_of_burst": achieved / pk["bf16_tflops"],
                "frac_of_sustained": achieved / pk["bf16_tflops_sustained"],
                "power_cap_active": "sw_power_cap" in (clocks or {}).get("reasons", []),
                "algorithmic_flops_per_launch": step_flops(cfg),
                "algorithmic_bytes_per_launch": step_bytes(cfg),
                "hbm_frac": step_bytes(cfg) / (kern_mean * 1e-3) / 1e9 / pk["hbm_gbs"],
                # secondary bound: one exponential per score element on the special-function unit
                # (16 per clock per SM, 148 SMs, at the SM clock sampled during the run)
                "sfu": sfu_bound(cfg, kern_mean, (clocks or {}).get("sm_mhz")),
            },
            "e2e": {"value": world * cfg.B * cfg.L * cfg.steps * e2e_blocks / (ms_e2e * 1e-3),
                    "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "blocks_timed": e2e_blocks},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "horizon": horizon_report(block_ms, mem_marks, layer.workspace_bytes + layer.state.numel() * 4),
            "commit_ms": commit_ms,
            "clean_pass_ms": clean_ms,
            # the commit is HBM-bound by its arithmetic intensity (about 175 flop/B); the same bytes
            # serve the delta and per-token-decay variants, whose extra work is on-chip
            "commit_roofline": {
                "bound": "hbm", "unit": "GB/s", "peak": pk["hbm_gbs"],
                "algorithmic_bytes": commit_bytes_flops(cfg)[0], "algorithmic_flops": commit_bytes_flops(cfg)[1],
                "achieved": {k: commit_bytes_flops(cfg)[0] / (v * 1e-3) / 1e9 for k, v in commit_ms.items()},
                "frac": {k: commit_bytes_flops(cfg)[0] / (v * 1e-3) / 1e9 / pk["hbm_gbs"] for k, v in commit_ms.items()},
            },
            "teacher_horizon": teacher,
            "batched_leg": batched,
            "chunked_leg": chunked,
            "module_stack": stack,
        }
        if world == 1 and not args.no_cpu_baseline:
            s = CpuSample(cfg)
            s.time_rows(s.threads)                      # the first call pays for page faults
            cal = 64 * s.threads
            t = s.time_rows(cal)
            n_rows = max(cal, int(cal * 15.0 / max(t, 1e-6)))   # about 15 s of CPU work
            tr = s.time_rows(n_rows)
            n_heads = min(s.threads, cfg.B * cfg.H)
            th = s.time_heads(n_heads)
            block_s = s.block_seconds(n_rows, tr, n_heads, th)
            line["cpu_baseline"] = {
                "value": cfg.B * cfg.L * cfg.steps / block_s, "unit": UNIT, "cores": s.threads,
                "kind": "oracle",
                "sample": (f"{n_rows} random output rows of one denoise pass ({tr:.1f} s) and the "
                           f"commit of {n_heads} heads ({th:.1f} s), extrapolated to one block"),
            }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long", choices=["tiny", "small", "chunked", "batched", "long"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-teacher", action="store_true", help="skip the teacher-attention horizon leg")
    ap.add_argument("--no-batched-leg", action="store_true", help="skip the short runs of the batched and chunked workloads")
    ap.add_argument("--no-stack", action="store_true", help="skip the 30-layer module stack leg")
    ap.add_argument("--traffic-probe", action="store_true",
                    help="set up, run four denoise passes and a commit, exit (for a one-launch profiler capture)")
    ap.add_argument("--probe-all", action="store_true",
                    help="with --traffic-probe: also call every other entry point once (bf16, D = 128)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return
    world = os.environ.get("WORLD_SIZE")
    if world is None and args.gpus > 1:
        # asked for N GPUs outside a launcher: start the N ranks here (one process per GPU)
        sys.exit(subprocess.call(launcher_command(args.gpus, sys.argv[1:])))
    if world is not None and int(world) != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started WORLD_SIZE={world} ranks")
    if args.traffic_probe:
        run_traffic_probe(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
