#!/usr/bin/env python
"""Benchmark of the LeanQuant per-linear-layer pass on B200.

A "step" is one pass of all four stages (Hessian, dampen/invert/factor, grid fit, column
loop) over one synthetic layer of the chosen workload.  Default workload: the
Llama-3-8B-shaped q_proj (W 4096 x 4096 bf16, X 4096 x 262144 bf16, 4-bit non-uniform,
p = 4, 20 k-means iterations, 128-column blocks).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun): every rank quantises its own layer (layers are independent
problems, no collective on the data path); value = weights of all ranks / max time.
--impl reference times the float64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

WORKLOADS = {
    # name: (recipe, r, c, n, settings)
    "llama3-8b-q_proj-nu4": ("c2", 4096, 4096, 262144, dict(grid="nonuniform", bits=4, p=4.0, n_iter=20)),
    "c1-512": ("c1", 512, 512, 8192, dict(grid="nonuniform", bits=4, p=4.0, n_iter=20)),
    # a quarter-size layer whose inputs (256 MiB of X) still exceed the L2: the case profiler captures run on
    "q_proj-2k-nu4": ("c2", 2048, 2048, 65536, dict(grid="nonuniform", bits=4, p=4.0, n_iter=20)),
    "aff-2k-g128": ("c3", 2048, 2048, 65536, dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9)),
    # a wide layer with little else to do: the case the stage-2 kernels are profiled on
    "wide-8k-nu4": ("c2", 512, 8192, 16384, dict(grid="nonuniform", bits=4, p=4.0, n_iter=20)),
    # the other benchmark configurations (parity-test cases; timed on request with --no-e2e --no-cpu-baseline)
    "llama3-8b-q_proj-nu3": ("c2", 4096, 4096, 262144, dict(grid="nonuniform", bits=3, p=4.0, n_iter=20)),
    # Eq. 7 at the paper's granularity (Appendix B: T = 2048, t = 0.2 T at 4 bits): 168100 candidates per group
    "aff-2k-g128-T2048": ("c3", 2048, 2048, 65536, dict(grid="affine", bits=4, p=4.0, group=128, T=2048, t=409)),
    "llama3-8b-q_proj-aff4row-T2048": ("c3", 4096, 4096, 262144, dict(grid="affine", bits=4, p=4.0, group=0, T=2048, t=409)),
    "llama3-8b-down_proj-aff4g128-T2048": ("c3", 4096, 14336, 131072,
                                           dict(grid="affine", bits=4, p=4.0, group=128, T=2048, t=409)),
    # Algorithm 2 (LeanQuant-Exact) on BERT-base-sized layers; a name ending in "-exact" selects lq_quantize_exact
    "bert-base-attn-768-nu4-exact": ("c2", 768, 768, 131072, dict(grid="nonuniform", bits=4, p=4.0, n_iter=20)),
    "bert-base-ffn_in-3072x768-nu3-exact": ("c2", 3072, 768, 131072, dict(grid="nonuniform", bits=3, p=4.0, n_iter=20)),
    "llama3-8b-down_proj-aff4g128": ("c3", 4096, 14336, 131072, dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9)),
    "llama3-8b-down_proj-nu3": ("c3", 4096, 14336, 131072, dict(grid="nonuniform", bits=3, p=4.0, n_iter=20)),
    "llama3-8b-gate_proj-nu3": ("c2", 14336, 4096, 131072, dict(grid="nonuniform", bits=3, p=4.0, n_iter=20)),
    "llama31-405b-up_proj-nu2": ("c3", 53248, 16384, 65536, dict(grid="nonuniform", bits=2, p=4.0, n_iter=20)),
    "llama31-405b-up_proj-aff4g128": ("c3", 53248, 16384, 65536, dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9)),
    "llama31-405b-down_proj-nu2": ("c3", 16384, 53248, 65536, dict(grid="nonuniform", bits=2, p=4.0, n_iter=20)),
    "llama31-405b-down_proj-aff4g128": ("c3", 16384, 53248, 65536, dict(grid="affine", bits=4, p=4.0, group=128, T=45, t=9)),
}
L2_BYTES = 126 * 1024 * 1024


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sust=p["bf16_tflops_sustained"], src="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sust=1400.0, src="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def layer_seed(rank: int) -> int:
    """Every rank quantises a different synthetic layer."""
    return 1000 + rank


def max_over_ranks(t: torch.Tensor, world: int) -> torch.Tensor:
    """Multi-rank timings are reported as the maximum over ranks."""
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ------------------------------------------------------------------ reference arm ----
def oracle_sample(name, seed=0, n_tokens=8192, n_rows=256, device="cpu", layer=None, c_sub=4096):
    """Times the float64 oracle on a bounded sample of the workload: stage 1 on `n_tokens`
    tokens (scaled up linearly), stage 2 in full, stages 3-4 on `n_rows` rows (scaled up
    linearly: rows are independent problems).  Layers wider than `c_sub` input features are
    sampled in that direction too: every stage runs on the first `c_sub` features and its time is
    scaled by its cost law in c (stage 1 c^2, stage 2 c^3, stage 3 c, stage 4 c^2), which makes
    the figure an extrapolation and is said so.  Returns (seconds for the full layer, description, cores)."""
    from oracle import leanquant_oracle as O
    recipe, r, c, n, st = WORKLOADS[name]
    exact = name.endswith("-exact")
    n_tokens = min(n_tokens, n)
    n_rows = min(n_rows, r, 4) if exact else min(n_rows, r)       # Algorithm 2 costs O(c^3) per row
    cs = min(c, c_sub)
    if st.get("group"):
        cs = cs // st["group"] * st["group"]
    if layer is None:
        layer = synth.make_layer(recipe, n_rows, cs, n_tokens, seed=seed, device=device)
        Xs = layer.X.double().cpu().numpy()
        Ws = layer.W.double().cpu().numpy()
    else:
        Xs = layer.X[:cs, :n_tokens].double().cpu().numpy()
        Ws = layer.W[:n_rows, :cs].double().cpu().numpy()
    fc = c / cs
    t0 = time.perf_counter()
    H = O.hessian(Xs)
    t1 = time.perf_counter()
    U, dinv, _, Wf = O.prepare_hinv(H, 0.01, Ws)
    t2 = time.perf_counter()
    s3_scale, s3_note = 1.0, ""
    if st["grid"] == "affine":
        # Eq. 7 costs (t + 1)^2 candidates per group: the search is timed on the first groups only, so that it stays
        # within ~10 s, and scaled up (groups are independent problems); the column loop then runs with those
        # parameters repeated over the row, which costs what the real ones cost
        g = st["group"] or cs
        ng = cs // g
        per_group = n_rows * g * (st["t"] + 1) ** 2 / 4e7                      # seconds, rough
        ng_s = int(max(1, min(ng, 10.0 / max(per_group, 1e-9))))
        S, Z = O.fit_grid_affine(Wf[:, :ng_s * g], dinv[:ng_s * g], st["bits"], st["p"], st["group"], st["T"], st["t"])
        t3 = time.perf_counter()
        s3_scale = ng / ng_s
        s3_note = f" (stage 3 on {ng_s} of {ng} groups per row, scaled x{s3_scale:g})"
        reps = -(-ng // ng_s)
        O.quantize_layer(Wf, U, scale=np.tile(S, (1, reps))[:, :ng], zero=np.tile(Z, (1, reps))[:, :ng], bits=st["bits"],
                         group=st["group"], block=128)
    else:
        G = O.fit_grid_nonuniform(Wf, dinv, st["bits"], st["p"], st["n_iter"])
        t3 = time.perf_counter()
        if exact:
            O.quantize_exact(Wf, U.T @ U, grid=G, bits=st["bits"])
        else:
            O.quantize_layer(Wf, U, grid=G, bits=st["bits"], block=128)
    t4 = time.perf_counter()
    full = ((t1 - t0) * (n / n_tokens) * fc ** 2 + (t2 - t1) * fc ** 3 +
            ((t3 - t2) * s3_scale * fc + (t4 - t3) * fc ** 2) * (r / n_rows))
    cores = len(os.sched_getaffinity(0))
    wide = "" if cs == c else (f"; all stages on the first {cs} of {c} input features, scaled by c^2 / c^3 / c / c^2 "
                               f"(x{fc ** 2:.3g} / x{fc ** 3:.3g} / x{fc:.3g} / x{fc ** 2:.3g})")
    desc = (f"float64 oracle: stage 1 on {n_tokens} of {n} tokens (scaled x{n / n_tokens:g}), stage 2 in full, "
            f"stages 3-4 on {n_rows} of {r} rows (scaled x{r / n_rows:g}){s3_note}{wide}; measured "
            f"{t1 - t0:.2f}+{t2 - t1:.2f}+{t3 - t2:.2f}+{t4 - t3:.2f} s, extrapolated to the full layer")
    return full, desc, cores


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    recipe, r, c, n, st = WORKLOADS[args.workload]
    times = []
    desc, cores = "", 0
    # every step is a bounded sample; with many steps the sample shrinks so that the run stays within minutes
    shrink = min(1.0, 4.0 / max(1, args.warmup + args.steps))
    ref_tokens = max(4096, int(args.ref_tokens * shrink) // 1024 * 1024)
    ref_rows = max(64, int(args.ref_rows * shrink) // 16 * 16)
    for i in range(args.warmup + args.steps):
        t, desc, cores = oracle_sample(args.workload, seed=i, n_tokens=ref_tokens, n_rows=ref_rows)
        if i >= args.warmup:
            times.append(t)
    sec = float(np.mean(times))
    val = r * c / sec
    line = {"impl": "reference", "metric": "weights quantized/sec per linear layer", "value": val,
            "unit": "weights/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": args.workload, "r": r, "c": c, "n_tokens": n, **st},
            "cpu_baseline": {"value": val, "unit": "weights/s", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": "weights/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------ our arm ----
def measure_pipes(lq, h, stream):
    """Rates of the plain arithmetic pipes on this GPU, from the library's dependent-free loops (CUDA events
    around one launch each, after a warm-up launch): fp32 lanes (T lane-op/s), fp64 FMA and fp64 MMA (TFLOP/s)."""
    out = {}
    for kind, iters in (("f32_fma", 1 << 15), ("f64_fma", 1 << 14), ("f64_mma", 1 << 12)):
        lq.lq_peak_probe(h, kind, 256)
        best = 0.0
        for _ in range(3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            ops = lq.lq_peak_probe(h, kind, iters)
            b.record(stream)
            torch.cuda.synchronize()
            best = max(best, ops / (a.elapsed_time(b) * 1e-3) / 1e12)
        out[kind] = best
    return out


def stage_rooflines(st, r, c, n, stage_ms, pk, pipes, w_bytes, exact=False):
    """Each stage's algorithmic work per second against the bound of the kernels that run it.
      stage 1: c^2 n flops (symmetry used) against the measured bf16 tensor peak (burst; sustained beside it);
      stage 2: 2/3 c^3 flops of the fused factorisation + inversion against the measured FP64 MMA rate;
      stage 3: Eq. 5: point-iterations x (log2 K + 3) fp32 lane-operations, Eq. 7: candidates x weights x 9, against
               the measured fp32 FMA lane rate; the one read of W against the measured HBM copy rate beside it;
      stage 4: the lazy updates' r c^2 flops against the bf16 tensor peak (`executed_frac` counts the bf16
               products actually issued per fp32 product)."""
    K = 1 << st["bits"]
    s1 = float(c) * c * n / (stage_ms[0] * 1e-3) / 1e12
    s2 = (2.0 / 3.0) * float(c) ** 3 / (stage_ms[1] * 1e-3) / 1e12
    if st["grid"] == "affine":
        s3_work = float(r) * c * (st["t"] + 1) ** 2 * 9
    else:
        s3_work = float(r) * c * st["n_iter"] * (np.log2(K) + 3)
    s3_ops = s3_work / (stage_ms[2] * 1e-3) / 1e12
    s3_exec = None
    if st["grid"] == "affine" and (st["t"] + 1) ** 2 >= 256 and st["T"] - 2 * st["t"] > 2 * (K - 1):
        # Fine partitions: the library scores one representative per class of candidates that give the same
        # grid (same t_min + t_max, same Z), eight lane-operations per weight; about this many per group:
        classes = sum((min(st["t"], u) - max(0, u - st["t"])) * (K - 1) / (st["T"] - u) + 1 for u in range(2 * st["t"] + 1))
        s3_exec = float(r) * c * classes * 8 / (stage_ms[2] * 1e-3) / 1e12
    s3_gbs = float(r) * c * w_bytes / (stage_ms[2] * 1e-3) / 1e9
    s4 = float(r) * c * c / (stage_ms[3] * 1e-3) / 1e12
    lane_peak, f64_peak = pipes["f32_fma"], pipes["f64_mma"]
    out = {
        "hessian": {"bound": "tensor", "achieved": s1, "peak": pk["tf_burst"], "unit": "TFLOP/s", "frac": s1 / pk["tf_burst"],
                    "frac_of_sustained": s1 / pk["tf_sust"]},
        "prepare_hinv": {"bound": "fp64 tensor", "achieved": s2, "peak": f64_peak, "unit": "TFLOP/s", "frac": s2 / f64_peak,
                         "peak_source": "measured: dependent-free mma.sync m8n8k4 f64 loop"},
        "fit_grid": {"bound": "alu", "achieved": s3_ops, "peak": lane_peak, "unit": "T lane-op/s", "frac": s3_ops / lane_peak,
                     "peak_source": "measured: dependent-free fp32 FMA loop",
                     "kind": "notional: the point-iterations of Eq. 5 (the candidate evaluations of Eq. 7) at their lane-operations each; "
                             "the k-means kernels sort or group a row once and then move K-1 boundaries on prefix sums, "
                             "so what binds them is latency (one warp per row runs the fp64 iterations), not this work",
                     "hbm_gbs": s3_gbs, "hbm_frac": s3_gbs / pk["hbm"],
                     "executed": s3_exec, "executed_frac": None if s3_exec is None else s3_exec / lane_peak},
        "quantize_layer": {"bound": "tensor", "achieved": s4, "peak": pk["tf_burst"], "unit": "TFLOP/s", "frac": s4 / pk["tf_burst"],
                           "executed_frac": STAGE4_PRODUCTS * s4 / pk["tf_burst"],
                           "executed_frac_of_sustained": STAGE4_PRODUCTS * s4 / pk["tf_sust"]},
    }
    dfrac = stage2_deferred_fraction(c)
    if dfrac > 0.0:
        # wide layers: most update products run on the integer tensor cores as 15 digit-slice products each, so the
        # algorithmic rate can exceed the FP64 pipe's peak; what the tensor pipe executes is reported beside it, against
        # the measured sustained bf16 rate times the nominal int8 / bf16 ratio (there is no measured int8 figure)
        ex = STAGE2_PRODUCTS * dfrac * s2
        out["prepare_hinv"].update({"bound": "tensor (int8 digit slices) for the deferred updates, fp64 tensor for the rest",
                                    "deferred_fraction": dfrac, "executed_int8_tops": ex,
                                    "int8_peak": INT8_OVER_BF16 * pk["tf_sust"],
                                    "executed_frac_of_sustained": ex / (INT8_OVER_BF16 * pk["tf_sust"])})
    if exact:
        # Algorithm 2: r rows x c steps x a c x c downdate = r c^3 fp64 FMAs, half of which touch weights already
        # quantised and need not be done
        s4x = 2.0 * float(r) * float(c) ** 3 / (stage_ms[3] * 1e-3) / 1e12
        out["quantize_layer"] = {"bound": "fp64 alu", "kernel": "exact_row_kernel (Algorithm 2)", "achieved": s4x,
                                 "peak": pipes["f64_fma"], "unit": "TFLOP/s", "frac": s4x / pipes["f64_fma"]}
    return out


STAGE4_PRODUCTS = 6     # bf16 products the library issues per fp32 product of the lazy update
STAGE2_PRODUCTS = 15    # 8-bit integer digit-slice products per fp64 product of stage 2's deferred updates
INT8_OVER_BF16 = 2.0    # nominal ratio of the dense int8 and bf16 tensor rates (4.5 vs 2.25 P op/s)
STAGE2_DEFER_MIN_BLOCKS, STAGE2_OUTER = 48, 8


def stage2_deferred_fraction(c):
    """Share of stage 2's update products (128 x 128 x 128 tile products) that the library defers to the bf16 tensor
    cores: it counts, step by step as the library's sweep goes, the tiles updated at once on the FP64 MMA (the rows
    and columns of the current outer block of 8 block columns) and the tiles that wait for the outer block's end."""
    nblk = -(-c // 128)
    if nblk < STAGE2_DEFER_MIN_BLOCKS:
        return 0.0
    eager = deferred = 0
    for o_lo in range(0, nblk, STAGE2_OUTER):
        o_hi = min(o_lo + STAGE2_OUTER, nblk) - 1
        for k in range(o_lo, o_hi + 1):
            for i in range(k):                       # block row i < k gets tiles j >= i
                n_all = nblk - i
                if i >= o_lo:
                    eager += n_all
                else:
                    n_in = o_hi - o_lo + 1           # columns of the outer block
                    eager += n_in
                    deferred += n_all - n_in
    return deferred / float(eager + deferred)


class LayerRun:
    """One single-layer workload on the device: inputs, buffers and the four calls."""

    def __init__(self, lq, h, name, dev, seed, chunk=0, layer=None, share=None):
        self.lq, self.h, self.name = lq, h, name
        recipe, r, c, n, st = WORKLOADS[name]
        self.r, self.c, self.n, self.st = r, c, n, st
        self.cfg = lq.Config.make(**st)
        self.layer = layer if layer is not None else synth.make_layer(recipe, r, c, n, seed=seed, device=dev)
        self.W, self.X = self.layer.W, self.layer.X
        self.chunk = n if chunk <= 0 else min(n, chunk)
        self.exact = name.endswith("-exact")
        self.share = share                                    # a LayerRun of the same layer whose stages 1-2 stand
        if share is None:
            self.P = lq.LayerPass(h, r, c, self.cfg, w_dtype=self.W.dtype, x_dtype=self.X.dtype, n_chunk=self.chunk, device=dev)
        else:
            self.P = lq.LayerPass.__new__(lq.LayerPass)
            self.P.__dict__.update(share.P.__dict__)
            self.P.cfg = self.cfg
            K = 1 << self.cfg.bits
            f32 = dict(device=dev, dtype=torch.float32)
            affine = st["grid"] == "affine"
            ng = 1 if not st.get("group") else c // st["group"]
            self.P.grid = None if affine else torch.empty((r, K), **f32)
            self.P.scale = torch.empty((r, ng), **f32) if affine else None
            self.P.zero = torch.empty((r, ng), device=dev, dtype=torch.int32) if affine else None
        self.ws_exact = (torch.empty(lq.lq_quantize_exact_workspace(self.cfg, r, c), dtype=torch.uint8, device=dev)
                         if self.exact else None)
        self.stream = torch.cuda.current_stream()

    def stage4(self, Wd, W_hat):
        lq, P = self.lq, self.P
        if self.exact:
            lq.lq_quantize_exact(self.h, self.cfg, Wd, P.U, P.codes, self.ws_exact, P.grid, P.scale, P.zero, W_hat, P.loss)
        else:
            lq.lq_quantize_layer(self.h, self.cfg, Wd, P.U, P.codes, P.ws, P.grid, P.scale, P.zero, W_hat, P.loss)

    def step(self, ev=None):
        lq, h, P, W, X, stream = self.lq, self.h, self.P, self.W, self.X, self.stream
        if self.share is None:
            P.H.zero_()
            if ev: ev[0].record(stream)
            for j in range(0, self.n, self.chunk):
                lq.lq_hessian_accumulate(h, X[:, j:j + self.chunk], P.H, 2.0, P.ws)
            if ev: ev[1].record(stream)
            lq.lq_hessian_finalize(h, P.H)
            lq.lq_prepare_hinv(h, P.H, P.U, P.dinv, P.ws, 0.01, W)
        elif ev:
            ev[0].record(stream)
            ev[1].record(stream)
        if ev: ev[2].record(stream)
        lq.lq_fit_grid(h, self.cfg, W, P.dinv, P.ws, P.grid, P.scale, P.zero)
        if ev: ev[3].record(stream)
        self.stage4(W, P.W_hat)
        if ev: ev[4].record(stream)

    def timed(self, steps, warmup, barrier=None, sampler=None):
        """`warmup` untimed steps, then `steps` timed ones between two synchronisations.  Returns (total ms,
        per-stage ms averaged over the steps, launches, clocks)."""
        lq = self.lq
        barrier = barrier or torch.cuda.synchronize
        for _ in range(warmup):
            self.step()
        lq.lq_sync_status(self.h)
        barrier()
        if sampler:
            sampler.start()
            time.sleep(0.25)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
        e_beg, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = lq.lq_launch_count()
        barrier()
        e_beg.record(self.stream)
        for i in range(steps):
            self.step(evs[i])
        e_end.record(self.stream)
        barrier()
        launches = lq.lq_launch_count() - launches0
        total_ms = e_beg.elapsed_time(e_end)
        clocks = sampler.stop() if sampler else None
        lq.lq_sync_status(self.h)
        stage_ms = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs]).mean(axis=0)
        return total_ms, stage_ms, int(launches), clocks


def extra_workloads(lq, h, dev, rank, pk, pipes, args):
    """The other benchmark configurations, each timed in this same run (3 warm-up + 3 timed steps, CUDA events):
    the 8B-shaped down_proj (affine g128, 100 candidates), the decoder block, and both 405B-shaped MLP layers
    (2-bit non-uniform and 4-bit affine g128; X passed in calls of 8192 tokens).  The affine variant of a 405B-shaped
    layer reuses the Hessian and factor of the non-uniform run of the same layer (its stages 1-2 are the same work,
    reported from that run); its stages 3-4 are timed on their own."""
    out = {}
    plan = [("llama3-8b-down_proj-aff4g128", 65536, None),
            ("llama3-8b-block-nu3", 0, None),
            ("llama31-405b-up_proj-nu2", 8192, None), ("llama31-405b-up_proj-aff4g128", 8192, "llama31-405b-up_proj-nu2"),
            ("llama31-405b-down_proj-nu2", 8192, None), ("llama31-405b-down_proj-aff4g128", 8192, "llama31-405b-down_proj-nu2")]
    steps, warmup = 3, 3
    prev = {}
    for name, chunk, share_name in plan:
        if args.only_workloads and name not in args.only_workloads:
            continue
        try:
            if name in BLOCKS:
                prev.clear()
                torch.cuda.empty_cache()
                out[name] = block_measure(lq, h, dev, rank, name, steps, warmup)
                torch.cuda.empty_cache()
                continue
            share = prev.get(share_name)
            if share is None:
                prev.clear()
                torch.cuda.empty_cache()
            run = LayerRun(lq, h, name, dev, layer_seed(rank), chunk, layer=share.layer if share else None, share=share)
            total_ms, stage_ms, launches, _ = run.timed(steps, warmup)
            if share is not None:
                stage_ms[0], stage_ms[1] = share.stage_ms[0], share.stage_ms[1]
                ms = float(stage_ms.sum())
            else:
                ms = total_ms / steps
            run.stage_ms = stage_ms
            r, c, n, st = run.r, run.c, run.n, run.st
            roofs = stage_rooflines(st, r, c, n, stage_ms, pk, pipes, run.W.element_size())
            entry = {"r": r, "c": c, "n_tokens": n, "tokens_per_call": run.chunk, **st, "steps": steps, "warmup": warmup,
                     "ms_per_step": ms, "value": r * c / (ms * 1e-3), "unit": "weights/s",
                     "stage_ms": {"hessian": float(stage_ms[0]), "prepare_hinv": float(stage_ms[1]),
                                  "fit_grid": float(stage_ms[2]), "quantize_layer": float(stage_ms[3])},
                     "stage_roofline_frac": {k: v["frac"] for k, v in roofs.items()},
                     "quantize_layer_executed_frac_of_sustained": roofs["quantize_layer"].get("executed_frac_of_sustained"),
                     "prepare_hinv_deferred_fraction": roofs["prepare_hinv"].get("deferred_fraction"),
                     "prepare_hinv_executed_int8_frac_of_sustained": roofs["prepare_hinv"].get("executed_frac_of_sustained"),
                     "gpu_launches_per_step": launches // steps}
            if share is not None:
                entry["note"] = f"stages 1-2 shared with {share_name} (same layer, same Hessian); their times are that run's"
            if not args.no_cpu_baseline:
                sec, desc, cores = oracle_sample(name, n_tokens=8192, n_rows=64, layer=run.layer, c_sub=2048)
                entry["cpu_baseline"] = {"value": r * c / sec, "unit": "weights/s", "cores": cores, "kind": "oracle",
                                         "sample": desc}
            out[name] = entry
            prev[name] = run
        except Exception as e:                                  # a workload that does not fit says so; the line still prints
            out[name] = {"error": f"{type(e).__name__}: {e}"}
            prev.clear()
            torch.cuda.empty_cache()
    prev.clear()
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import paper_2407_10032_b200 as lq
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    h = lq.lq_create(local)
    run = LayerRun(lq, h, args.workload, dev, layer_seed(rank), args.chunk)
    r, c, n, st, chunk = run.r, run.c, run.n, run.st, run.chunk
    W, X, P, cfg, layer, stream = run.W, run.X, run.P, run.cfg, run.layer, run.stream

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    total_ms, stage_ms, launches, clocks = run.timed(args.steps, args.warmup, barrier, sampler)

    # ---- end to end through the public API with host buffers -------------------------------
    e2e_ms, h2d, d2h = float("nan"), 0, 0
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, 3))
        # calibration activations on the host as they are collected: contiguous chunks of tokens, pinned
        e2e_chunk = min(chunk, 32768)
        Xh = []
        for j in range(0, n, e2e_chunk):
            t = torch.empty((c, min(e2e_chunk, n - j)), dtype=X.dtype, pin_memory=True)
            t.copy_(X[:, j:j + e2e_chunk])
            Xh.append(t)
        Wh = torch.empty(W.shape, dtype=W.dtype, pin_memory=True)
        Wh.copy_(W)
        outs = [t for t in (P.codes, P.grid, P.scale, P.zero, P.loss) if t is not None]
        outs_h = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs]
        Wd = torch.empty_like(W)

        def e2e_step():
            Wd.copy_(Wh, non_blocking=True)
            P.H.zero_()
            P.accumulate_from_host(Xh)                   # chunk copies overlapped with the contraction
            lq.lq_hessian_finalize(h, P.H)
            lq.lq_prepare_hinv(h, P.H, P.U, P.dinv, P.ws, 0.01, Wd)
            lq.lq_fit_grid(h, cfg, Wd, P.dinv, P.ws, P.grid, P.scale, P.zero)
            run.stage4(Wd, None)
            for th, td in zip(outs_h, outs):
                th.copy_(td, non_blocking=True)

        e2e_step()                                       # one untimed step: staging buffers, side stream and events exist after it
        barrier()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        b1.record(stream)
        barrier()
        e2e_ms = b0.elapsed_time(b1) / e2e_steps
        h2d = sum(t.numel() * t.element_size() for t in Xh) + Wh.numel() * Wh.element_size()
        d2h = sum(t.numel() * t.element_size() for t in outs_h)
        del Xh, Wh, Wd

    t = max_over_ranks(torch.tensor([total_ms, e2e_ms], device=dev, dtype=torch.float64), world)
    total_ms, e2e_ms = float(t[0]), float(t[1])
    ms_per_step = total_ms / args.steps
    weights = r * c * world
    value = weights / (ms_per_step * 1e-3)

    if rank == 0:
        pk = peaks()
        pipes = measure_pipes(lq, h, stream)
        # Dominant kernel (largest share of the step, see profiles/launch_list_*): the stage-1 tensor-core
        # contraction.  Algorithmic work with the symmetry used: c^2 * n flops (n tokens, c(c+1)/2 outputs,
        # 2 flops each).  `traffic` is the DRAM read+write byte count of that launch from a profiler capture
        # (dram__bytes_read.sum + dram__bytes_write.sum); it is only valid for the workload it was taken on.
        flops = float(c) * c * n
        ach = flops / (stage_ms[0] * 1e-3) / 1e12
        peak = pk["tf_burst"]
        traffic = 4777421056 if args.workload == "llama3-8b-q_proj-nu4" else None      # dram read + write of this launch, one ncu capture (it varies with how far the CTA pairs drift apart: 4.8 - 7.7 GB seen)
        roof = {"bound": "tensor", "kernel": "lq_tc_gemm_kernel (stage 1, H += 2XX^T)", "achieved": ach, "peak": peak,
                "unit": "TFLOP/s", "frac": ach / peak, "traffic": traffic, "peak_source": pk["src"] + " burst bf16",
                "frac_of_sustained": ach / pk["tf_sust"], "flops_per_launch": flops,
                "algorithmic_bytes_per_launch": 2.0 * c * n + 4.0 * c * c}
        stage_roof = stage_rooflines(st, r, c, n, stage_ms, pk, pipes, W.element_size(), run.exact)
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            sec, desc, cores = oracle_sample(args.workload, n_tokens=args.ref_tokens, n_rows=args.ref_rows, layer=layer)
            cpu = {"value": r * c / sec, "unit": "weights/s", "cores": cores, "kind": "oracle", "sample": desc}
        line = {
            "metric": "weights quantized/sec per linear layer", "value": value, "unit": "weights/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": args.workload, "r": r, "c": c, "n_tokens": n, "tokens_per_call": chunk, **st, "block": 128,
                       "damp": 0.01,
                       "l2": f"inputs per step ({(X.numel() * X.element_size()) >> 20} MiB X) exceed the 126 MiB L2",
                       "parallelism": "one layer per GPU, no collective",
                       "headline": "benchmark configuration 2 (the 8B-shaped q_proj at the paper's 262144 calibration tokens), the "
                                   "layer the metric is quoted on; the other configurations are under `workloads`"},
            "stage_ms": {"hessian": float(stage_ms[0]), "prepare_hinv": float(stage_ms[1]),
                         "fit_grid": float(stage_ms[2]), "quantize_layer": float(stage_ms[3])},
            "roofline": roof, "stage_roofline": stage_roof, "measured_pipes": pipes, "cpu_baseline": cpu,
            "e2e": None if args.no_e2e else {"value": weights / (e2e_ms * 1e-3), "unit": "weights/s",
                                             "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": int(launches), "clocks": clocks,
        }
        if world == 1 and not args.no_workloads:
            del run, P, W, X, layer
            torch.cuda.empty_cache()
            line["workloads"] = extra_workloads(lq, h, dev, rank, pk, pipes, args)
        print(json.dumps(line))
    lq.lq_destroy(h)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------- a whole decoder block ----
# Benchmark config 4: the seven linear layers of one Llama-3-8B-shaped decoder block, 3-bit non-uniform,
# n = 131072 tokens.  Layers that read the same activations share stages 1-2 (one Hessian for q/k/v, one for o,
# one for gate/up, one for down), which is how a model-level driver would call the library.
BLOCKS = {
    "llama3-8b-block-nu3": dict(
        n=131072, settings=dict(grid="nonuniform", bits=3, p=4.0, n_iter=20),
        inputs=[("attn_in", 4096, "c2", [("q_proj", 4096), ("k_proj", 1024), ("v_proj", 1024)]),
                ("o_in", 4096, "c2", [("o_proj", 4096)]),
                ("mlp_in", 4096, "c2", [("gate_proj", 14336), ("up_proj", 14336)]),
                ("down_in", 14336, "c3", [("down_proj", 4096)])]),
}


def block_measure(lq, h, dev, rank, name, steps, warmup):
    """Times the decoder-block workload through the library's stack driver (StackPass: layers in order, stages 1-2 once
    per distinct input, a packed record per layer); returns the fields of its report."""
    spec = BLOCKS[name]
    n, st = spec["n"], spec["settings"]
    cfg = lq.Config.make(**st)
    stream = torch.cuda.current_stream()
    inputs, weights, names = [], [], []
    for gi, (gname, c, recipe, layers) in enumerate(spec["inputs"]):
        Ws = []
        for li, (lname, r) in enumerate(layers):
            layer = synth.make_layer(recipe, r, c, n if li == 0 else 256, seed=layer_seed(rank) + 16 * gi + li, device=dev)
            if li == 0:
                inputs.append(layer.X)
            Ws.append(layer.W)
            del layer
        weights.append(Ws)
        names.append("hessian+prepare:" + gname)
        names.extend(l[0] for l in layers)
    S = lq.StackPass(h, [(c, [r for _, r in layers]) for _, c, _, layers in spec["inputs"]], cfg, w_dtype=weights[0][0].dtype,
                     x_dtype=inputs[0].dtype, n_chunk=n, device=dev, want_w_hat=False, want_records=True)

    def one_step(events=None):
        k = [0]

        def mark(g, l):
            if events:
                events[k[0]].record(stream)
                k[0] += 1
        S.run(inputs, weights, on_layer=mark)

    n_ev = len(names)
    for _ in range(warmup):
        one_step()
    lq.lq_sync_status(h)
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(steps)]
    e_beg, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = lq.lq_launch_count()
    torch.cuda.synchronize()
    e_beg.record(stream)
    for i in range(steps):
        one_step(evs[i])
    e_end.record(stream)
    torch.cuda.synchronize()
    launches = lq.lq_launch_count() - launches0
    total_ms = e_beg.elapsed_time(e_end)
    lq.lq_sync_status(h)
    parts = {}
    for j, nm in enumerate(names):
        beg = [e_beg if (i == 0 and j == 0) else (evs[i - 1][-1] if j == 0 else evs[i][j - 1]) for i in range(steps)]
        parts[nm] = float(np.mean([beg[i].elapsed_time(evs[i][j]) for i in range(steps)]))
    weights_n = sum(W.numel() for Ws in weights for W in Ws)
    payload_bits = sum(W.numel() * lq.lq_pack_layer_bytes(cfg, W.shape[0], W.shape[1])[1] for Ws in weights for W in Ws)
    ms_per_step = total_ms / steps
    return {"weights": weights_n, "n_tokens": n, **st, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step,
            "value": weights_n / (ms_per_step * 1e-3), "unit": "weights/s",
            "sharing": "stages 1-2 once per distinct input (4 Hessians for 7 layers)", "part_ms": parts,
            "record_bits_per_weight": payload_bits / weights_n,
            "gpu_launches_per_step": int(launches) // steps}


def run_block(args):
    import paper_2407_10032_b200 as lq
    rank, world, local = dist_env()
    if world > 1:
        raise SystemExit("bench.py: the block workload runs on one GPU")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    h = lq.lq_create(local)
    sampler = ClockSampler(local)
    sampler.start()
    m = block_measure(lq, h, dev, rank, args.workload, args.steps, args.warmup)
    clocks = sampler.stop()
    st = BLOCKS[args.workload]["settings"]
    print(json.dumps({
        "metric": "weights quantized/sec per linear layer", "value": m["value"], "unit": "weights/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": m["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "weights": m["weights"], "n_tokens": m["n_tokens"], **st, "block": 128, "damp": 0.01,
                   "sharing": m["sharing"], "l2": "each Hessian input (1 to 3.8 GB) exceeds the 126 MiB L2"},
        "part_ms": m["part_ms"], "roofline": None, "cpu_baseline": None, "e2e": None,
        "gpu_launches": m["gpu_launches_per_step"] * args.steps, "clocks": clocks}))
    lq.lq_destroy(h)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3-8b-q_proj-nu4", choices=sorted(WORKLOADS) + sorted(BLOCKS))
    ap.add_argument("--ref-tokens", type=int, default=65536)
    ap.add_argument("--ref-rows", type=int, default=1024)
    ap.add_argument("--chunk", type=int, default=0, help="tokens per Hessian call (0 = all at once)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (e2e is then null)")
    ap.add_argument("--no-cpu-baseline", action="store_true",
                    help="skip the oracle timing leg (profiler captures only; cpu_baseline is then null)")
    ap.add_argument("--no-workloads", action="store_true",
                    help="time the headline workload only (the `workloads` object of the other configurations is left out)")
    ap.add_argument("--only-workloads", nargs="*", default=None, help="restrict the `workloads` object to these names")
    args = ap.parse_args()
    if args.workload != "llama3-8b-q_proj-nu4":
        args.no_workloads = True                       # the other configurations ride on the default line only
    if args.workload in BLOCKS:
        if args.impl == "reference":
            raise SystemExit("bench.py: the block workload has no reference arm; use a single-layer workload")
        run_block(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
