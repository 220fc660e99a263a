"""Benchmark of the verify-and-judge step (aj_verify) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|sweep] [--impl reference]

A step is one whole cycle (LM-head projection + argmax, then judge + prefix scan: two launches) over one
batch of seeded synthetic inputs shaped like the paper's Llama-3.x pairs.  The headline workload is
the batch-1 8B-shaped configuration (B=1, K=16, d=4096, V=128256, bf16), the setting the paper's own
measurements use (batch size 1); the batched 8B- and 70B-shaped configurations, four points of the sweep
around the HBM / tensor crossover, and two variants of the acceptance step (sampled target tokens, the top-K
rule) are reported under "extra" in the same JSON line.  Metric: verified draft positions per second (B*K per cycle).

Rank layout for N > 1: one process per GPU, every rank verifies its own batch against its own copy
of W_lm (sequences are independent, there is no data-path collective): weak scaling.
With --sharding vocab the LM head is instead split by vocabulary over the ranks, all ranks verify the
SAME batch and exchange their per-row keys inside the kernels (peer stores over NVLink): strong scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import aj_inputs as gen  # noqa: E402

METRIC = "verified_positions_per_s"
UNIT = "positions/s"
L2_BYTES = 126 * 1024 * 1024


def workload(name: str) -> gen.Config:
    return {"c2": gen.C2, "c3": gen.C3, "c4": gen.C4}[name]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------ clocks


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20", "-i", str(self.gpu)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def wait_first(self, timeout: float = 4.0):
        """nvidia-smi takes a few hundred milliseconds to print its first row: wait for it, so that a
        timed region that starts now falls inside the sampled time."""
        t = time.time()
        while self.proc and not self.rows and time.time() - t < timeout and self.proc.poll() is None:
            time.sleep(0.01)

    def __exit__(self, *exc):
        if self.proc:
            time.sleep(0.03)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        rows = [r for t, r in self.rows if t0 <= t <= t1 and len(r) >= 7] or [r for _, r in self.rows if len(r) >= 7]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        sm = [float(r[0]) for r in rows]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].lower().startswith("active") for r in rows)]
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(rows[0][1]), "power_w_max": max(float(r[2]) for r in rows),
                "samples": len(rows), "reasons": reasons}


# ------------------------------------------------------------------------------- our GPU arm


class GpuWorkload:
    """One workload resident on the device: rotating copies of W_lm, inputs, outputs, handles."""

    def __init__(self, cfg: gen.Config, device: int, w_copies: int, W_host=None, flags: int = 0, group=None, rule=None):
        import torch

        import paper_2504_20039_b200 as aj

        self.torch, self.aj, self.cfg = torch, aj, cfg
        dev = f"cuda:{device}"
        bf = lambda a: torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
        W_host = gen.make_W(cfg) if W_host is None else W_host
        self.exchanges = []
        self.v_count = cfg.V
        shard = [None, None]
        if group is not None:  # vocabulary-parallel: this rank keeps only its rows of W_lm
            from paper_2504_20039_b200 import dist as ajd

            v0, vn = aj.shard_range(cfg.V, group.info.world, group.info.rank)
            W_host = W_host[v0 : v0 + vn]
            self.v_count = vn
            for i in range(2):  # one set of exchange buffers per handle: each handle counts its own cycles
                ex = ajd.Exchange(group, cfg.B, cfg.K)
                self.exchanges.append(ex)
                shard[i] = (group.info.rank, group.info.world, v0, vn, ex.buffers)
        self.W = [bf(W_host)]
        for _ in range(w_copies - 1):
            self.W.append(self.W[0].clone())
        ht, hd = gen.make_hidden(cfg)
        self.ht_host, self.hd_host = ht, hd
        self.ht, self.hd = bf(ht), bf(hd)
        self.w = torch.from_numpy(gen.make_judge(cfg)).to(dev)
        i32 = dict(dtype=torch.int32, device=dev)
        self.acc = torch.empty(cfg.B, **i32)
        self.nxt = torch.empty(cfg.B, **i32)
        self.tt = torch.empty((cfg.B, cfg.K + 1), **i32)
        self.handle = aj.Handle(device, cfg.B, cfg.K, cfg.d, cfg.d_draft, cfg.V, aj.AJ_BF16, aj.AJ_W_VD, flags, shard=shard[0])
        self.handle_t = aj.Handle(device, cfg.B, cfg.K, cfg.d, cfg.d_draft, cfg.V, aj.AJ_BF16, aj.AJ_W_VD,
                                  flags | aj.AJ_FLAG_TIME_KERNELS, shard=shard[1])
        for h in (self.handle, self.handle_t):  # the variants of the acceptance step: top-K rule, sampled target tokens
            if rule and rule.get("fuse_judge"):
                h.fuse_judge(self.w, stream=torch.cuda.current_stream().cuda_stream)
            if rule and rule.get("top_k"):
                h.set_top_k(rule["top_k"])
            if rule and rule.get("temperature"):
                from paper_2504_20039_b200 import dist as ajd_

                rk = int(os.environ.get("RANK", "0"))
                h.set_sampling(rule["temperature"], seed=ajd_.sampling_seed(20250420, rk, "vocab" if group is not None else "batch"), step=0)
        for ex in self.exchanges:
            ex.ready()
        # draft tokens planted against the device's own greedy tokens (a benchmark input, never an oracle input)
        self.tok = torch.from_numpy(gen.random_draft_tokens(cfg)).to(dev)
        self.step(self.handle, 0)
        torch.cuda.synchronize()
        self.tok_host = gen.plant_draft_tokens(cfg, self.tt.cpu().numpy())
        self.tok = torch.from_numpy(self.tok_host).to(dev)
        self.i = 0

    def step(self, handle, i):
        cfg = self.cfg
        handle.verify(self.ht, self.hd, self.W[i % len(self.W)], self.tok, self.w, cfg.judge_b, cfg.tau, cfg.B, cfg.K,
                      self.acc, self.nxt, self.tt, stream=self.torch.cuda.current_stream().cuda_stream)

    def run(self, handle, steps):
        for _ in range(steps):
            self.step(handle, self.i)
            self.i += 1

    def timed(self, handle, steps, barrier):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda.synchronize()
        t0 = time.time()
        e0.record()
        self.run(handle, steps)
        e1.record()
        torch.cuda.synchronize()
        t1 = time.time()
        barrier()
        return e0.elapsed_time(e1), t0, t1

    def e2e(self, steps, warmup):
        """The same cycle through aj_verify_host: per-cycle tensors start in pinned host memory."""
        torch, cfg = self.torch, self.cfg
        pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
        ht, hd, tok = pin(self.ht_host), pin(self.hd_host), pin(self.tok_host)
        acc = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        nxt = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        stream = torch.cuda.current_stream().cuda_stream
        call = lambda i: self.handle.verify_host(ht, hd, self.W[i % len(self.W)], tok, self.w, cfg.judge_b, cfg.tau, cfg.B, cfg.K,
                                                 acc, nxt, None, stream=stream)
        for i in range(warmup):
            call(i)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(steps):
            call(i)  # synchronous: returns when accept_len / next_tok are on the host
        dt = time.perf_counter() - t0
        h2d = ht.numel() * 2 + hd.numel() * 2 + tok.numel() * 4
        d2h = 8 * cfg.B
        return dt / steps, h2d, d2h

    def close(self):
        self.torch.cuda.synchronize()
        for ex in self.exchanges:
            ex.close()
        self.handle.destroy()
        self.handle_t.destroy()


# DRAM traffic per launch of the projection kernel (dram__bytes_read.sum + dram__bytes_write.sum of one
# profiler capture each), kept as data next to the capture summaries.  A figure is reported only while
# the kernel's sources still hash to what was captured.
CSRC = os.path.join(ROOT, "paper_2504_20039_b200", "csrc")
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")


def _traffic_table():
    try:
        with open(TRAFFIC_FILE) as f:
            return {(e["workload"], e["kernel"]): (float(e["bytes_per_launch"]), e["sources"], e["sources_sha1_12"]) for e in json.load(f)["captures"]}
    except (OSError, ValueError, KeyError):
        return {}


def _sources_sha(files):
    import hashlib

    h = hashlib.sha1()
    for f in files:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def traffic_of(cfg: gen.Config, path: str):
    ent = _traffic_table().get((cfg.name, path))
    if not ent:
        return None
    byts, files, sha = ent
    try:
        return byts if _sources_sha(files) == sha else None
    except OSError:
        return None


def roofline_of(cfg: gen.Config, gemm_ms: float, pk, v_count=None, gemm_ms_min=None, step_ms=None, alone_ms=None):
    """Roofline of the projection kernel: W streamed once from HBM vs 2*M*d*V flops on the tensor pipe
    (V = the vocabulary entries this GPU projects).  gemm_ms is the kernel's mean duration inside the
    timed loop (CUDA events around the launch); gemm_ms_min its shortest launch, what the kernel does
    before the power cap pulls the clock down (the peaks are burst figures of the same kind);
    step_ms the whole cycle measured in the same pass, for a fraction of the cycle, not of the kernel."""
    V = cfg.V if v_count is None else v_count
    flops = 2.0 * cfg.M * cfg.d * V
    byts = 2.0 * cfg.d * V + 2.0 * cfg.M * cfg.d + 8.0 * cfg.M
    t_hbm = byts / (pk["hbm_gbs"] * 1e9)
    t_tc = flops / (pk["bf16_tflops"] * 1e12)
    s = gemm_ms * 1e-3
    if t_hbm >= t_tc:
        a = byts / s / 1e9
        r = {"bound": "hbm", "achieved": a, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": a / pk["hbm_gbs"],
             "traffic": None, "peak_source": f"of {pk['source']}", "kernel_ms": gemm_ms, "algorithmic_bytes": byts}
    else:
        a = flops / s / 1e12
        r = {"bound": "tensor", "achieved": a, "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": a / pk["bf16_tflops"],
             "frac_of_sustained_peak": a / pk["bf16_tflops_sustained"], "sustained_peak": pk["bf16_tflops_sustained"],
             "peak_kind": "burst; kernel_ms is the mean launch of a loop that runs under the power cap, for which the sustained "
                          "peak is the like-for-like figure (frac_of_sustained_peak); frac_alone is the launch timed alone against the burst peak",
             "traffic": None, "peak_source": f"of {pk['source']}",
             "kernel_ms": gemm_ms, "algorithmic_flops": flops}
    t_roof = max(t_hbm, t_tc)
    r["roofline_ms"] = t_roof * 1e3
    if gemm_ms_min:
        r["kernel_ms_min"] = gemm_ms_min
        r["frac_shortest_launch"] = t_roof / (gemm_ms_min * 1e-3)
    if alone_ms:
        r["kernel_ms_alone"] = alone_ms  # best of 10 single launches after 50 ms of idle: comparable with the burst peak
        r["frac_alone"] = t_roof / (alone_ms * 1e-3)
    if step_ms:
        r["cycle_ms_same_pass"] = step_ms  # this pass records two events per cycle, which lengthens a cycle a little
    return r


MAX_REGIONS = 200  # --max-regions


def bench_one(cfg, device, steps, warmup, barrier, reduce_max, pk, w_copies, W_host=None, with_e2e=True, flags=0, group=None, rule=None):
    wl = GpuWorkload(cfg, device, w_copies, W_host, flags, group, rule)
    try:
        with ClockSampler(device) as cs:
            cs.wait_first()
            wl.run(wl.handle, warmup)
            # First a pass with events around the projection kernel (ring of 512 launches); the cycle time of
            # THIS pass is reported beside the kernel time, since the event records lengthen a cycle a little
            # and the two passes are separate measurements.  It runs before the main pass, not after it:
            # after 0.35 s at the power cap the part is hotter and the same kernel measures a few per cent slower.
            wl.run(wl.handle_t, min(warmup, 8))
            wl.handle_t.gemm_ms_stats()
            prof_steps = min(max(steps, 64), 512)
            pass_ms, t_begin, t_end = wl.timed(wl.handle_t, prof_steps, barrier)
            gemm_mean, gemm_min, n = wl.handle_t.gemm_ms_stats()
            # The timed region is exactly `steps` cycles.  A short region (20 cycles of 160 us) ends before
            # the clock sampler's first tick and is noisy, so it is repeated, every repeat bracketed by its
            # own events, until about 0.35 s have been timed; the median region is reported.
            first, _, t_end = wl.timed(wl.handle, steps, barrier)
            regions = [reduce_max(first)]
            repeats = int(min(MAX_REGIONS, max(1, -(-350.0 // max(regions[0], 1e-3)))))
            for _ in range(repeats - 1):
                ms_r, _, t_end = wl.timed(wl.handle, steps, barrier)
                regions.append(reduce_max(ms_r))
        clocks = cs.summary(t_begin, t_end)
        # the kernel timed alone, the way the burst peak it is compared with was taken (best of 10 single
        # launches, the GPU left idle for 50 ms before each so that the clock is not held down by the power cap)
        burst = []
        for i in range(10):
            torch_sync = wl.torch.cuda.synchronize
            torch_sync()
            time.sleep(0.05)
            wl.step(wl.handle_t, i)
            torch_sync()
            burst.append(wl.handle_t.last_gemm_ms())
        wl.handle_t.gemm_ms_stats()
        ms = statistics.median(regions)
        assert wl.handle.last_status() == wl.aj.AJ_OK and wl.handle_t.last_status() == wl.aj.AJ_OK
        res = {
            "ms_per_step": ms / steps, "clocks": clocks, "path": wl.handle.last_gemm_path(),
            "timing": {"regions_of_steps": len(regions), "ms_per_step_min": min(regions) / steps, "ms_per_step_max": max(regions) / steps,
                       "reported": "median region"},
            "roofline": dict(roofline_of(cfg, gemm_mean, pk, wl.v_count, gemm_min, pass_ms / prof_steps, min(burst)),
                             traffic=None if (group is not None or rule) else traffic_of(cfg, wl.handle.last_gemm_path())),
            "gemm_ms_min": gemm_min, "gemm_launches_timed": n,
            "launches_per_step": wl.handle.last_launch_count(),
            "mean_accept_len": float(wl.acc.float().mean().item()),
        }
        # the whole cycle (both kernels, as timed in the main pass) against the same roofline
        res["roofline"]["frac_whole_cycle"] = res["roofline"]["roofline_ms"] / res["ms_per_step"]
        if with_e2e:
            s, h2d, d2h = wl.e2e(max(10, min(steps, 300)), 5)
            res["e2e_s_per_step"] = reduce_max(s)
            res["h2d"], res["d2h"] = h2d, d2h
        return res
    finally:
        wl.close()


def cpu_baseline(cfg: gen.Config, W_host=None, budget_s: float = 12.0):
    """The CPU oracle, as it stands, on a bounded sample of the workload: whole sequences (K+1 rows
    against the full vocabulary), one per pass, cycling through the batch until about `budget_s`
    seconds of CPU work have been timed (at least one pass)."""
    from oracle import aj_oracle as orc

    sub = gen.scaled(cfg, B=1)
    W = gen.make_W(cfg) if W_host is None else W_host
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    tok = gen.random_draft_tokens(sub)
    passes, dt, r = 0, 0.0, None
    while passes == 0 or dt < budget_s:
        b = passes % cfg.B
        t0 = time.perf_counter()
        r = orc.verify(ht[b : b + 1], None if hd is None else hd[b : b + 1], W, tok, w, cfg.judge_b, cfg.tau, cfg.dtype)
        dt += time.perf_counter() - t0
        passes += 1
    return {"value": passes * cfg.K / dt, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{passes} passes of one whole sequence each ({cfg.K + 1} rows x V={cfg.V}, d={cfg.d}; batch of {cfg.B}), "
                      f"{dt:.1f} s of fp64 loops"}, r


def reference_arm(args):
    """--impl reference: the CPU oracle timed on the host cores (there is no other reference program)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import aj_oracle as orc

    cfg = workload(args.workload if args.workload not in ("sweep", "lr_fit") else "c2")
    steps = args.steps if args.steps is not None else 3
    warmup = args.warmup if args.warmup is not None else 1
    W = gen.make_W(cfg)
    for _ in range(warmup):
        cpu_baseline(cfg, W, budget_s=0.0)
    t0 = time.perf_counter()
    for _ in range(steps):
        base, _ = cpu_baseline(cfg, W, budget_s=0.0)  # one pass = one whole sequence per step
    dt = (time.perf_counter() - t0) / steps
    value = cfg.K / dt  # one sequence per step
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": cfg.name, "B": 1, "K": cfg.K, "d": cfg.d, "d_draft": cfg.d_draft, "V": cfg.V,
                                       "note": "each step verifies one whole sequence of the workload with the CPU oracle"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": base["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def lr_fit_line(args):
    """The classifier fit at the paper's training-set size (Section 4.1: about 130 K mined mismatches, 20 %
    important; features [h_draft ; h_target] of the 1B / 8B pair; C = 1e-4): whole fits timed with CUDA events,
    HBM roofline of the loss + gradient kernel from its share of the fit (one pass over X per evaluation)."""
    import torch

    import paper_2504_20039_b200 as aj

    if int(os.environ.get("RANK", "0")) != 0:
        return
    n, F, C = 131072, 6144, 1e-4
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    g = torch.Generator(device=dev).manual_seed(20250420)
    X = torch.empty((n, F), dtype=torch.bfloat16, device=dev)
    u = torch.randn(F, generator=g, device=dev)
    u /= u.norm()
    score = torch.empty(n, device=dev)
    for i in range(0, n, 8192):  # unit Gaussians, labelled by a noisy projection: the top 20 % are "important"
        blk = torch.randn((min(8192, n - i), F), generator=g, device=dev)
        X[i : i + blk.shape[0]] = blk.to(torch.bfloat16)
        score[i : i + blk.shape[0]] = X[i : i + blk.shape[0]].float() @ u
    score += torch.randn(n, generator=g, device=dev)
    y = (score > torch.quantile(score[:: max(1, n // 65536)], 0.8)).to(torch.uint8)
    w = torch.zeros(F, dtype=torch.float32, device=dev)
    steps = args.steps if args.steps is not None else 3
    warmup = args.warmup if args.warmup is not None else 1
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(warmup):
        aj.lr_fit(0, X, y, n, F, aj.AJ_BF16, C, w, stream=stream)
    pk = peaks()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(0) as cs:
        torch.cuda.synchronize()
        t0 = time.time()
        e0.record()
        evals, kernel_ms = 0, 0.0
        for _ in range(steps):
            st, b, iters, ev, gnorm = aj.lr_fit(0, X, y, n, F, aj.AJ_BF16, C, w, stream=stream)
            evals += ev
            kernel_ms += aj.lr_fit.kernel_ms
        e1.record()
        torch.cuda.synchronize()
        t1 = time.time()
    ms = e0.elapsed_time(e1)
    byts = float(n) * F * 2
    per_eval_s = kernel_ms * 1e-3 / evals  # the loss + gradient kernel alone (CUDA events inside the library)
    line = {
        "metric": "lr_fit_rows_per_s", "value": n * evals / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1, "steps": steps, "warmup": warmup,
        "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 features, fp32 accumulate, fp64 optimiser",
        "data": "synthetic", "config": {"workload": "lr_fit_131072x6144", "n": n, "F": F, "C": C, "iterations": iters, "evaluations_per_fit": evals // steps,
                                          "max_abs_gradient": gnorm, "intercept": b, "positives": float(y.float().mean().item()),
                                          "l2": "X is 1.61 GB, larger than the 126 MB L2"},
        "clocks": cs.summary(t0, t1),
        "roofline": {"bound": "hbm", "achieved": byts / per_eval_s / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": byts / per_eval_s / 1e9 / pk["hbm_gbs"], "traffic": None, "peak_source": f"of {pk['source']}",
                     "kernel_ms": kernel_ms / evals, "note": "the loss + gradient kernel, one pass over X per evaluation; a whole fit also allocates its workspace, copies w down and the gradient up per evaluation and runs L-BFGS on the host",
                     "algorithmic_bytes": byts},
        "gpu_launches": 2 * evals, "e2e": None,
    }
    if not args.no_cpu:
        from oracle import aj_lr_oracle as lro

        rows = 4096
        Xs = X[:rows].float().cpu().numpy().astype(np.float64)
        ys = y[:rows].cpu().numpy()
        wz = np.zeros(F)
        t = time.time()
        passes = 0
        while time.time() - t < 10.0:
            lro.objective(Xs, ys, C, wz, 0.0)
            passes += 1
        dt = time.time() - t
        line["cpu_baseline"] = {"value": rows * passes / dt, "unit": "rows/s", "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"{passes} evaluations of the objective and its gradient on the first {rows} rows (fp64 numpy)"}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "sweep", "lr_fit"])
    ap.add_argument("--point", default=None, metavar="BxK", help="one point of the sweep on the 8B shape as the workload, e.g. 8x32")
    ap.add_argument("--max-regions", type=int, default=200, help="most repeats of the timed region (1 for profiler captures)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the batched configurations reported under 'extra'")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer (end-to-end) measurement; for profiler captures")
    ap.add_argument("--sharding", default="batch", choices=["batch", "vocab"],
                    help="batch: every rank its own batch and its own W_lm (default); vocab: W_lm split by vocabulary over the ranks")
    ap.add_argument("--flags", type=int, default=0, help="extra aj_create flags (kernel selection switches, for comparisons)")
    ap.add_argument("--top-k", type=int, default=0, help="time the top-K acceptance rule (paper Section 4.1) instead of the classifier")
    ap.add_argument("--temperature", type=float, default=0.0, help="time sampled verification (paper Appendix A) at this temperature instead of greedy")
    ap.add_argument("--fuse-judge", action="store_true", help="compute the classifier's target half inside the projection kernel (paper Section 3.2)")
    ap.add_argument("--w-copies", type=int, default=None, help="copies of W_lm to rotate over (default 3, or 2 for the 70B shape)")
    args = ap.parse_args()
    if args.impl == "reference":
        return reference_arm(args)
    if args.workload == "lr_fit":
        return lr_fit_line(args)

    import torch

    from paper_2504_20039_b200 import dist as ajd

    info = ajd.rank_info()
    rank, world, local = info.rank, info.world, info.local_rank
    torch.cuda.set_device(local)
    group = ajd.Group(info, backend="nccl", device=torch.device(f"cuda:{local}"))
    barrier, reduce_max = group.barrier, group.max_over_ranks

    global MAX_REGIONS
    MAX_REGIONS = max(1, args.max_regions)
    pk = peaks()
    head = workload("c2" if args.workload == "sweep" else args.workload)
    if args.point:
        head = gen.sweep_config(*map(int, args.point.lower().split("x")))
    default_steps = {"c2": 4000, "c3": 400, "c4": 200, "c5": max(20, int(0.4 / max(2.0 * head.M * head.d * head.V / 1.2e15, 1.7e-4)))}[head.name[:2]]
    steps = args.steps if args.steps is not None else default_steps
    warmup = max(3, args.warmup if args.warmup is not None else 10)
    copies = args.w_copies or (3 if head.d * head.V * 2 < 1.5e9 else 2)

    vocab = args.sharding == "vocab"
    rule = {k: v for k, v in (("top_k", args.top_k), ("temperature", args.temperature), ("fuse_judge", args.fuse_judge)) if v}
    if not vocab:
        head = ajd.rank_config(head, rank)  # every rank verifies its own sequences
    W_host = gen.make_W(head)
    r = bench_one(head, local, steps, warmup, barrier, reduce_max, pk, copies, W_host, with_e2e=not args.no_e2e, flags=args.flags,
                  group=group if vocab else None, rule=rule)
    positions = head.B * head.K if vocab else ajd.job_positions(head, world)
    line = {
        "metric": METRIC, "value": positions / (r["ms_per_step"] * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": r["ms_per_step"], "us_per_cycle": r["ms_per_step"] * 1e3, "higher_is_better": True,
        "scaling": "strong" if vocab else "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": head.name, "B": head.B, "K": head.K, "d": head.d, "d_draft": head.d_draft, "V": head.V,
                   "tau": head.tau, "match_rate": [head.match_lo, head.match_hi], "parallelism": (f"W_lm split by vocabulary over {world} GPU(s), one batch, keys exchanged by peer stores inside the kernels"
                                   if vocab else f"replicated W, batch per rank x{world}"),
                   "l2": f"W_lm rotates over {copies} copies of {head.d * head.V * 2 / 1e9:.2f} GB each (inputs larger than the 126 MB L2)",
                   "gemm_path": r["path"], "mean_accept_len": r["mean_accept_len"],
                   "rule": rule or "classifier at tau on greedy target tokens"},
        "clocks": r["clocks"], "roofline": r["roofline"], "timing": r["timing"],
        "gpu_launches": r["launches_per_step"] * steps,
    }
    if "e2e_s_per_step" in r:
        line["e2e"] = {"value": positions / r["e2e_s_per_step"], "unit": UNIT, "h2d_bytes_per_step": r["h2d"],
                       "d2h_bytes_per_step": r["d2h"], "us_per_cycle": r["e2e_s_per_step"] * 1e6,
                       "note": "aj_verify_host: hidden states copied from pinned host memory, draft tokens read and results "
                               "written in place over PCIe by the judge kernel; W_lm and judge_w are resident parameters"}

    extra = []
    if not args.no_extra:
        todo = []
        if args.workload == "sweep":
            todo = [gen.sweep_config(B, K) for B in gen.SWEEP_B for K in gen.SWEEP_K]
        elif args.workload == "c2" and not vocab and not args.point:
            # the batched 8B- and 70B-shaped workloads, and the four points of the sweep around the crossover
            # from HBM-bound to tensor-bound (136, 264, 520 and 576 rows)
            todo = [gen.C3, gen.sweep_config(8, 16), gen.sweep_config(8, 32), gen.sweep_config(8, 64), gen.sweep_config(64, 8), gen.C4]
            if not rule:
                # and the two variants of the acceptance step whose epilogues do more, each right after the
                # default rule on the same workload: sampled target tokens at C3, the top-K rule at C4
                todo = [gen.C3, (gen.C3, {"temperature": 1.0})] + todo[1:] + [(gen.C4, {"top_k": 8})]
        for item in todo:
            cfg, item_rule = item if isinstance(item, tuple) else (item, rule)
            cfg = ajd.rank_config(cfg, rank)
            same_W = cfg.d == head.d and cfg.V == head.V
            n = max(20, int(0.4 / max(2.0 * cfg.M * cfg.d * cfg.V / 1.2e15, 1.7e-4)))
            rr = bench_one(cfg, local, n, 5, barrier, reduce_max, pk, 2 if not same_W else copies, W_host if same_W else None, with_e2e=False, flags=args.flags, rule=item_rule)
            extra.append({"workload": cfg.name, "B": cfg.B, "K": cfg.K, "d": cfg.d, "V": cfg.V, "steps": n,
                          "ms_per_step": rr["ms_per_step"], "value": cfg.B * cfg.K * world / (rr["ms_per_step"] * 1e-3), "unit": UNIT,
                          "gemm_path": rr["path"], "rule": item_rule or "classifier at tau on greedy target tokens",
                          "roofline": rr["roofline"], "clocks": rr["clocks"]})
    if world > 1 and not vocab and args.workload == "c2" and not args.no_extra:
        # Strong scaling of the headline workload with the LM head split by vocabulary over the ranks: one batch,
        # every rank streams 1/N of W_lm, per-row keys exchanged by peer stores inside the kernels.  Recorded
        # beside the replicas above so that a multi-GPU run exercises the exchange; a failure here is reported,
        # not fatal (set-up fails on every rank or on none).
        c2 = gen.C2
        try:
            rr = bench_one(c2, local, steps, warmup, barrier, reduce_max, pk, copies, W_host if (c2.d, c2.V, c2.seed) == (head.d, head.V, head.seed) else None,
                           with_e2e=False, flags=args.flags, group=group, rule=rule)
            extra.append({"workload": c2.name, "sharding": "vocab", "scaling": "strong", "n_gpus": world, "B": c2.B, "K": c2.K, "steps": steps,
                          "ms_per_step": rr["ms_per_step"], "value": c2.B * c2.K / (rr["ms_per_step"] * 1e-3), "unit": UNIT,
                          "gemm_path": rr["path"], "roofline": rr["roofline"], "clocks": rr["clocks"], "timing": rr["timing"],
                          "parallelism": f"W_lm split by vocabulary over {world} GPUs, one batch, keys exchanged by peer stores inside the kernels"})
        except Exception as e:  # noqa: BLE001
            extra.append({"workload": c2.name, "sharding": "vocab", "n_gpus": world, "error": repr(e)[:300]})
    line["extra"] = extra

    if rank == 0 and world == 1 and not args.no_cpu:
        base, _ = cpu_baseline(head, W_host)
        line["cpu_baseline"] = base
    if rank == 0:
        print(json.dumps(line))
    group.close()


if __name__ == "__main__":
    main()
