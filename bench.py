#!/usr/bin/env python
"""Benchmark of the folded-MoE layer (ExFold hot path) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload glm45air|mixtral|qwen3|tiny] [--k-pre K'] [--pool-m M] ...

One step = one pass of the whole hot path: a prefill call over T tokens (token-level Top-K'
folding) followed by a decode call over a batch of B tokens (pool-M folding), on seeded
synthetic inputs shaped like the named model. Prints ONE JSON line (rank 0):
  value        prefill tokens/s of the whole job, inputs resident in HBM (device-timed, max over ranks)
  decode       microseconds per decode layer and its HBM roofline
  e2e          the same metric through the host-buffer entry points (pinned host x/logits in, y out)
  roofline     dominant prefill kernel (grouped GEMM-1) against the measured bf16 tensor peak
  cpu_baseline the CPU oracle timed on this machine's host cores on a bounded sample (rank 0, N=1)
  sustained    the headline prefill call back to back for >= 2 s against the sustained bf16 peak
  configs      the same measurements for every other benchmark configuration (N=1, no --workload):
               Mixtral-shaped, Qwen3-shaped (K' = 4 and 6, M = 16/32/64), tiny fp32, and the
               batch x pool decode sweep on the Qwen3 shape
Without --workload the headline is the largest single-GPU configuration (GLM-4.5-Air-shaped) and
`configs` carries the rest; with --workload only that layer is measured (profiling, reduced cases).
With N > 1 (torchrun) every rank runs an independent replica of the headline layer: the path has no
exchange step, so there is no collective on the data path.
--impl reference times the CPU oracle alone (there is no reference implementation to install).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

HEADLINE = "glm45air"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}  # the figures the benchmark spec names
# DRAM bytes measured by ncu (dram__bytes_read.sum + dram__bytes_write.sum) divided by the algorithmic
# bytes of the same launch, from the reduced-case ncu captures whose summaries are under profiles/
# (same rows per expert as the full-size workload, fewer experts or a shorter intermediate size so that
# the capture stays small). Traffic grows with the weights, so the full-size figure is this ratio times
# the full-size algorithmic bytes. A shape without a capture reports traffic = null.
NCU_TRAFFIC_RATIO = {
    # profiles/kernels_mixtral_reduced.md, kernels_qwen3_full.md, kernels_glm45air_reduced.md
    "mixtral": {"gemm1": 426.8 / 318.8, "decode_ffn": 138.6 / 134.7},
    "qwen3": {"gemm1": 899.7 / 820.0, "decode_ffn": 105.0 / 101.7},
    "glm45air": {"gemm1": 1343.2 / 986.7, "decode_ffn": 771.6 / 765.6},
}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period: float = 0.004):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML missing: report that instead of clocks
            self.err = repr(e)

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80, "sync_boost": 0x10}
        while not self.stop_flag.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self.stop_flag.set()
        self.join()
        return self.summary()

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "note": "no NVML samples"}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def build_inputs(cfg, T, B):
    t0 = time.time()
    inp = dict(x=si.hidden_states(cfg, T), lg=si.router_logits(cfg, T), xd=si.hidden_states(cfg, B, "x_dec"),
               lgd=si.router_logits(cfg, B, "logits_dec"))
    inp["wg"], inp["wu"], inp["wd"] = si.expert_weights(cfg)
    inp["tables"] = si.synthetic_tables(cfg)
    log(f"[bench] {cfg.name}: inputs generated in {time.time() - t0:.1f}s")
    return inp


def oracle_sample_run(cfg, inp, Kp, n_tokens, seed=7):
    """CPU oracle on a seeded sample of prefill tokens (routing at full size)."""
    import oracle
    A = si.as_oracle_array
    S, L, h, lnh = [t.numpy() for t in inp["tables"]]
    T = inp["x"].shape[0]
    n = min(n_tokens, T)
    idx = np.sort(np.random.default_rng(seed).choice(T, size=n, replace=False)).astype(np.int64)
    t0 = time.perf_counter()
    fold = oracle.prefill_fold(inp["lg"].numpy(), cfg.top_k, Kp, S, L, h, lnh)
    t_fold = time.perf_counter() - t0
    t0 = time.perf_counter()
    y = oracle.moe_apply(A(inp["x"]), A(inp["wg"]), A(inp["wu"]), A(inp["wd"]), fold["ids"], fold["w"],
                         cfg.n_experts, cfg.n_shared, tok_idx=idx)
    t_apply = time.perf_counter() - t0
    sec = t_apply + t_fold * n / T
    return dict(idx=idx, y=y, fold=fold, seconds=sec, tokens=n, tokens_per_s=n / sec)


def oracle_decode_run(cfg, inp, M):
    import oracle
    A = si.as_oracle_array
    S, L, h, lnh = [t.numpy() for t in inp["tables"]]
    t0 = time.perf_counter()
    dec = oracle.decode_fold(inp["lgd"].numpy(), cfg.top_k, M, S, L, h)
    y = oracle.moe_apply(A(inp["xd"]), A(inp["wg"]), A(inp["wu"]), A(inp["wd"]), dec["ids"], dec["w"], cfg.n_experts,
                         cfg.n_shared)
    return dict(dec=dec, y=y, seconds=time.perf_counter() - t0)


def max_over_ranks(values, world, device="cpu"):
    """Element-wise MAX of a list of floats over all ranks (the slowest rank defines the job's time)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_tokens_per_s(tokens_per_rank, world, ms):
    """Whole-job throughput of `world` independent replicas that each process tokens_per_rank tokens in ms."""
    return world * tokens_per_rank / (ms * 1e-3)


def rel_err(y, ref):
    return float(np.abs(y - ref).max() / np.abs(ref).max()), float(np.linalg.norm(y - ref) / np.linalg.norm(ref))


def r4(v):
    """Round to 5 significant digits (keeps the JSON line short)."""
    if v is None:
        return None
    return float(f"{float(v):.5g}")


def workload_config(args, name=None):
    cfg = si.CONFIGS[name or args.workload or HEADLINE]
    over = {}
    if args.tokens:
        over["prefill_tokens"] = args.tokens
    if args.batch:
        over["decode_batch"] = args.batch
    if args.inter:
        over["inter"] = args.inter
    if args.experts:
        over["n_experts"] = args.experts
    if over:
        cfg = si.scaled(cfg, name=cfg.name + "-reduced", **over)
    return cfg


class Flush:
    """Evicts L2 between calls by READING a 512 MiB buffer: the cache is left full of clean lines.
    (Writing the buffer instead would leave ~126 MB of dirty lines whose write-back is then charged to
    the first reads of the timed kernel: about 20 us of foreign DRAM traffic per call.)"""

    def __init__(self, dev):
        import torch
        self.torch = torch
        self.buf = torch.zeros(128 << 20, dtype=torch.int32, device=dev)  # 512 MiB, > 4x L2

    def __call__(self):
        self.torch.sum(self.buf)


class Workload:
    """One synthetic layer resident on the device, with the calls the benchmark times."""

    def __init__(self, ex, cfg, dev, batches=None):
        import torch
        self.ex, self.cfg, self.dev, self.torch = ex, cfg, dev, torch
        self.T, self.B = cfg.prefill_tokens, cfg.decode_batch
        maxB = max([self.B] + list(batches or []))
        self.inp = build_inputs(cfg, self.T, maxB)
        g = lambda t: t.to(dev)
        inp = self.inp
        self.x, self.lg = g(inp["x"]), g(inp["lg"])
        self.xd_all, self.lgd_all = g(inp["xd"]), g(inp["lgd"])
        self.wg, self.wu, self.wd = g(inp["wg"]), g(inp["wu"]), g(inp["wd"])
        self.tabs = [g(t) for t in inp["tables"]]
        self.tables = ex.make_tables(*self.tabs)
        self.layer = ex.make_layer(cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.inter, cfg.top_k, cfg.dtype)
        self.ws = ex.alloc_workspace(self.layer, max(self.T, maxB), cfg.top_k, host_staging=True)
        self.y = torch.empty((self.T, cfg.hidden), dtype=self.wg.dtype, device=dev)
        self.el = 2 if cfg.dtype == "bf16" else 4
        self.set_batch(self.B)

    def set_batch(self, B):
        torch = self.torch
        self.B = B
        self.xd, self.lgd = self.xd_all[:B].contiguous(), self.lgd_all[:B].contiguous()
        self.yd = torch.empty((B, self.cfg.hidden), dtype=self.wg.dtype, device=self.dev)
        self.dmeta = dict(pool_size=torch.zeros(1, dtype=torch.int32, device=self.dev))

    def prefill(self, Kp, meta=None):
        self.ex.exfold_moe_prefill(self.layer, self.x, self.lg, self.wg, self.wu, self.wd, self.tables, Kp, self.y,
                                   self.ws, meta=meta)

    def decode(self, M):
        self.ex.exfold_moe_decode(self.layer, self.xd, self.lgd, self.wg, self.wu, self.wd, self.tables, M, self.yd,
                                  self.ws, meta=self.dmeta)

    def status_ok(self, what):
        assert self.ex.exfold_device_status(self.ws) == 0, f"device status after {what}"

    def timed(self, fn, steps, warmup, flush):
        """Per-call CUDA events on the launching stream, L2 evicted before every call. Returns ms per call."""
        torch = self.torch
        for _ in range(warmup):
            flush()
            fn()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush()
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]

    def kernel_times(self, fn, reps, flush):
        ex, torch = self.ex, self.torch
        ex.exfold_profile_enable(True)
        kern = {}
        for _ in range(reps):
            flush()
            fn()
            torch.cuda.synchronize()
            for k_, v in ex.exfold_profile_read().items():
                kern.setdefault(k_, []).append(v)
        ex.exfold_profile_enable(False)
        return {k_: float(np.mean(v)) for k_, v in kern.items()}

    def free(self):
        for k in list(self.__dict__):
            if k not in ("torch",):
                self.__dict__.pop(k)
        self.torch.cuda.empty_cache()


def prefill_report(wl, Kp, ms_list, kern, peaks, peak_src, world=1):
    """Fractions for one prefill configuration. Algorithmic work: 6 d I flop per (token, executed expert);
    compulsory HBM bytes: every touched expert's weights once + x + y + logits."""
    import torch
    cfg = wl.cfg
    T, N, d, I, el = wl.T, cfg.n_experts, cfg.hidden, cfg.inter, wl.el
    ms = float(np.mean(ms_list))
    rows = T * Kp + T * cfg.n_shared
    flop = rows * 6.0 * d * I
    off = torch.zeros(N + 1, dtype=torch.int32, device=wl.dev)
    wl.prefill(Kp, meta=dict(offsets=off))
    torch.cuda.synchronize()
    touched = int((np.diff(off.cpu().numpy()) > 0).sum()) + cfg.n_shared
    byts = touched * 3.0 * d * I * el + 2.0 * T * d * el + 4.0 * T * N
    t_c, t_m = flop / (peaks["bf16_tflops"] * 1e12) * 1e3, byts / (peaks["hbm_gbs"] * 1e9) * 1e3
    out = {"k_pre": Kp, "ms": r4(ms), "ms_min": r4(np.min(ms_list)), "tokens_per_s": r4(world * T / (ms * 1e-3)),
           "useful_tflops": r4(flop / (ms * 1e-3) / 1e12),
           "frac_of_bf16_peak": r4(flop / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]),
           "frac_of_bf16_sustained": r4(flop / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]),
           "frac_of_nominal_bf16": r4(flop / (ms * 1e-3) / 1e12 / NOMINAL["bf16_tflops"]),
           "touched_experts": touched, "t_compute_ms": r4(t_c), "t_hbm_ms": r4(t_m),
           "frac_of_bound": r4(max(t_c, t_m) / ms), "flop": flop, "compulsory_bytes": byts}
    if kern:
        out["kernels_ms"] = {k: r4(v) for k, v in kern.items()}
        if "gemm1_gateup_swiglu" in kern:
            f1, f2 = rows * 4.0 * d * I, rows * 2.0 * d * I
            out["gemm1_frac"] = r4(f1 / (kern["gemm1_gateup_swiglu"] * 1e-3) / 1e12 / peaks["bf16_tflops"])
            out["gemm2_frac"] = r4(f2 / (kern["gemm2_down_combine"] * 1e-3) / 1e12 / peaks["bf16_tflops"])
            out["non_gemm_ms"] = r4(sum(v for k, v in kern.items() if k in ("prefill_route", "prefill_scatter",
                                                                            "convert_bf16")))
    return out


def prefill_roofline(wl, Kp, kern, peaks, peak_src, touched):
    cfg = wl.cfg
    T, d, I, el = wl.T, cfg.hidden, cfg.inter, wl.el
    rows = T * Kp + T * cfg.n_shared
    if "gemm1_gateup_swiglu" in kern:
        f1 = rows * 4.0 * d * I
        ach = f1 / (kern["gemm1_gateup_swiglu"] * 1e-3) / 1e12
        b1 = touched * 2.0 * d * I * el + rows * d * el + rows * I * el
        ratio = NCU_TRAFFIC_RATIO.get(cfg.name.replace("-reduced", ""), {}).get("gemm1")
        return {"kernel": "grouped GEMM-1 (gate/up + SwiGLU), tcgen05", "bound": "tensor", "achieved": r4(ach),
                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": r4(ach / peaks["bf16_tflops"]),
                "traffic": None if ratio is None else b1 * ratio,
                "traffic_note": "ncu reduced-case DRAM bytes / algorithmic bytes x full-size algorithmic bytes"
                                if ratio else "no ncu capture of this shape",
                "peak_source": f"{peak_src} burst bf16 matmul", "launch_ms": r4(kern["gemm1_gateup_swiglu"]),
                "flop_per_launch": f1, "algorithmic_bytes_per_launch": b1}
    if "simt_ffn" in kern:
        flop = rows * 6.0 * d * I
        ach = flop / (kern["simt_ffn"] * 1e-3) / 1e12
        return {"kernel": "SIMT fp32 expert FFN", "bound": "alu", "achieved": r4(ach), "peak": 72.0,
                "unit": "TFLOP/s", "frac": r4(ach / 72.0), "traffic": None, "launch_ms": r4(kern["simt_ffn"]),
                "flop_per_launch": flop, "peak_source": "148 SMs x 128 fp32 lanes x 2 flop x 1.9 GHz"}
    return None


def decode_report(wl, M, ms_list, kern, peaks, static_ms=None):
    cfg = wl.cfg
    d, I, el = cfg.hidden, cfg.inter, wl.el
    ms = float(np.mean(ms_list))
    pool = int(wl.dmeta["pool_size"].item())
    byts = (pool + cfg.n_shared) * 3.0 * d * I * el
    gbs = byts / (ms * 1e-3) / 1e9
    out = {"batch": wl.B, "pool_m": M, "effective_pool": pool, "us_per_layer": r4(ms * 1e3),
           "us_min": r4(np.min(ms_list) * 1e3), "pool_weight_bytes": byts, "gbs_on_pool_bytes": r4(gbs),
           "frac_of_measured_hbm": r4(gbs / peaks["hbm_gbs"]), "frac_of_8tbs": r4(gbs / NOMINAL["hbm_gbs"])}
    if static_ms is not None:
        out["static_pool_us_per_layer"] = r4(float(np.mean(static_ms)) * 1e3)
    if kern:
        out["kernels_ms"] = {k: r4(v) for k, v in kern.items()}
    return out


def decode_roofline(wl, kern, peaks, pool):
    cfg = wl.cfg
    byts = (pool + cfg.n_shared) * 3.0 * cfg.hidden * cfg.inter * wl.el
    name = cfg.name.replace("-reduced", "")
    if "decode_ffn" in kern:  # gate/up kernel (routing prologue + the pool's gate and up weights, x read in place)
        gu = byts * 2.0 / 3.0
        t = kern["decode_ffn"] * 1e-3
        ratio = NCU_TRAFFIC_RATIO.get(name, {}).get("decode_ffn")
        out = {"kernel": "decode gate/up kernel (pool / remap prologue + gate and up weight stream over the pool), tcgen05",
               "bound": "hbm", "achieved": r4(gu / t / 1e9), "peak": peaks["hbm_gbs"], "unit": "GB/s",
               "frac": r4(gu / t / 1e9 / peaks["hbm_gbs"]), "traffic": None if ratio is None else gu * ratio,
               "bytes_per_launch": gu, "launch_ms": r4(kern["decode_ffn"])}
        td = kern.get("decode_down", 0.0) * 1e-3
        if td > 0:
            out["down_gbs"] = r4(byts / 3.0 / td / 1e9)
            out["ffn_gbs"] = r4(byts / (t + td) / 1e9)
        return out
    if "decode_gateup" in kern:
        gu = byts * 2.0 / 3.0
        tg = kern["decode_gateup"] * 1e-3
        ratio = NCU_TRAFFIC_RATIO.get(name, {}).get("decode_gateup")
        out = {"kernel": "decode GEMM-1 (gate/up weight stream over the pool), tcgen05", "bound": "hbm",
               "achieved": r4(gu / tg / 1e9), "peak": peaks["hbm_gbs"], "unit": "GB/s",
               "frac": r4(gu / tg / 1e9 / peaks["hbm_gbs"]), "traffic": None if ratio is None else gu * ratio,
               "bytes_per_launch": gu, "launch_ms": r4(kern["decode_gateup"])}
        td = kern.get("decode_down", 0.0) * 1e-3
        if td > 0:
            out["down_gbs"] = r4(byts / 3.0 / td / 1e9)
            out["ffn_gbs"] = r4(byts / (tg + td) / 1e9)
        return out
    return None


def e2e_leg(wl, Kp, M, reps, flush, world=1):
    """Through the host-buffer entry points: pinned host x / logits in, y out, copies inside the timed region."""
    torch, ex, cfg = wl.torch, wl.ex, wl.cfg
    inp, T, B, d, N = wl.inp, wl.T, wl.B, cfg.hidden, cfg.n_experts
    xh, lh = inp["x"].pin_memory(), inp["lg"].pin_memory()
    xdh, ldh = inp["xd"][:B].contiguous().pin_memory(), inp["lgd"][:B].contiguous().pin_memory()
    yh = torch.empty((T, d), dtype=wl.wg.dtype).pin_memory()
    ydh = torch.empty((B, d), dtype=wl.wg.dtype).pin_memory()
    ee = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(reps)]
    for it in range(reps + 2):
        k = max(it - 2, 0)
        flush()
        ee[k][0].record()
        ex.exfold_moe_prefill_host(wl.layer, xh, lh, wl.wg, wl.wu, wl.wd, wl.tables, Kp, yh, wl.ws)
        ee[k][1].record()
        flush()
        ee[k][2].record()
        ex.exfold_moe_decode_host(wl.layer, xdh, ldh, wl.wg, wl.wu, wl.wd, wl.tables, M, ydh, wl.ws)
        ee[k][3].record()
        torch.cuda.synchronize()
    pre = float(np.mean([e[0].elapsed_time(e[1]) for e in ee]))
    dec = float(np.mean([e[2].elapsed_time(e[3]) for e in ee]))
    pre, dec = max_over_ranks([pre, dec], world, wl.dev)
    el = wl.el
    return {"value": r4(job_tokens_per_s(T, world, pre)), "unit": "tokens/s",
            "h2d_bytes_per_step": int(T * d * el + T * N * 4 + B * d * el + B * N * 4),
            "d2h_bytes_per_step": int(T * d * el + B * d * el), "prefill_ms": r4(pre), "decode_us": r4(dec * 1e3)}


def cpu_baseline_leg(wl, Kp, M, flop_budget):
    """The oracle as it stands on a bounded sample of the same workload; the sample doubles as a parity check
    of the benchmarked outputs (wl.y / wl.yd must hold the results of prefill(Kp) / decode(M))."""
    import oracle
    cfg = wl.cfg
    d, I, K = cfg.hidden, cfg.inter, cfg.top_k
    per_tok = (Kp + cfg.n_shared) * 6.0 * d * I
    n_s = int(max(1, min(2048, flop_budget / per_tok)))
    t0 = time.time()
    o = oracle_sample_run(cfg, wl.inp, Kp, n_s)
    yg = wl.y.float().cpu().numpy()[o["idx"]]
    emax, efro = rel_err(yg, o["y"])
    base = {"value": r4(o["tokens_per_s"]), "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{o['tokens']} seeded prefill tokens (all their routes) of the same workload; routing at "
                      f"full size; {o['seconds']:.1f}s"}
    parity = {"prefill_max_err_rel": r4(emax), "prefill_fro_err_rel": r4(efro), "tokens": int(o["tokens"])}
    if wl.B * (K + cfg.n_shared) * 6.0 * d * I <= 4 * flop_budget:
        inp = dict(wl.inp)
        inp["xd"], inp["lgd"] = wl.inp["xd"][:wl.B], wl.inp["lgd"][:wl.B]
        od = oracle_decode_run(cfg, inp, M)
        dmax, dfro = rel_err(wl.yd.float().cpu().numpy(), od["y"])
        base["decode_us_per_layer"] = r4(od["seconds"] * 1e6)
        parity.update({"decode_max_err_rel": r4(dmax), "decode_fro_err_rel": r4(dfro)})
    log(f"[bench] {cfg.name}: cpu baseline took {time.time() - t0:.1f}s")
    return base, parity


def static_pool_for(wl, M):
    torch, ex, cfg = wl.torch, wl.ex, wl.cfg
    i32 = dict(dtype=torch.int32, device=wl.dev)
    keep = (torch.empty(M, **i32), torch.empty(cfg.n_experts, **i32),
            torch.empty(cfg.n_experts, dtype=torch.float32, device=wl.dev))
    sp = ex.exfold_static_pool_build(wl.layer, wl.tables, M, *keep)
    return sp, keep


def stack_leg(wl, M, L, flush, Kp=None, reps=8):
    """L layers of the workload's shape run one after the other on one stream, each = router scores (W_r x) + folded
    layer, every layer with its own weights (device views rolled along the expert axis, so no weight line is reused
    between layers) and router matrix, layer l+1 reading layer l's output. Timed as plain stream launches and as one
    captured CUDA graph. Kp = None: decode layers on the decode batch; else prefill layers on the prefill tokens."""
    torch, ex, cfg = wl.torch, wl.ex, wl.cfg
    N, d = cfg.n_experts, cfg.hidden
    per = [(torch.roll(wl.wg, l, 0), torch.roll(wl.wu, l, 0), torch.roll(wl.wd, l, 0)) if l else (wl.wg, wl.wu, wl.wd)
           for l in range(L)]
    wr0 = si.router_weights(cfg).to(wl.dev)
    wrs = [torch.roll(wr0, l, 0) for l in range(L)]
    x0 = wl.xd if Kp is None else wl.x
    n = x0.shape[0]
    lgs = [torch.empty((n, N), dtype=torch.float32, device=wl.dev) for _ in range(L)]
    hs = [x0] + [torch.empty((n, d), dtype=wl.wg.dtype, device=wl.dev) for _ in range(L)]

    def run_layers():
        for l in range(L):
            if Kp is None:
                ex.exfold_moe_decode_layer(wl.layer, hs[l], wrs[l], per[l][0], per[l][1], per[l][2], wl.tables, M,
                                           hs[l + 1], wl.ws, logits_out=lgs[l])
            else:
                ex.exfold_moe_prefill_layer(wl.layer, hs[l], wrs[l], per[l][0], per[l][1], per[l][2], wl.tables, Kp,
                                            hs[l + 1], wl.ws, logits_out=lgs[l])

    def timed(fn):
        ts = []
        for it in range(reps + 2):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    res = {"layers": L, "mode": "decode" if Kp is None else "prefill",
           "what": "router scores + folded layer per layer, own weights per layer, each layer reads the previous output"}
    res["stream_us_per_layer"] = r4(timed(run_layers) * 1e3 / L)
    wl.status_ok("the layer stack")
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            run_layers()
        torch.cuda.synchronize()
        res["graph_us_per_layer"] = r4(timed(graph.replay) * 1e3 / L)
        wl.status_ok("the graph replays")
    except Exception as e:  # capture is an optional measurement: report, do not lose the benchmark line
        res["graph_error"] = f"{type(e).__name__}: {e}"[:300]
    return res


def measure_config(ex, cfg, dev, args, peaks, peak_src, flush, steps, warmup, with_cpu=True, with_e2e=True,
                   sweep=None, stack_layers=0):
    """All measurements of one configuration, device-timed at N=1: every K' of the config for prefill, every M for
    decode (dynamic pool, and the static pool beside it), per-kernel times, fractions, e2e and the CPU baseline of
    the config's first (K', M)."""
    torch = __import__("torch")
    wl = Workload(ex, cfg, dev, batches=sweep[0] if sweep else None)
    rec = {"workload": describe(cfg), "dtype": cfg.dtype, "prefill": [], "decode": []}
    for Kp in cfg.k_pre:
        ms = wl.timed(lambda: wl.prefill(Kp), steps, warmup, flush)
        kern = wl.kernel_times(lambda: wl.prefill(Kp), min(steps, 6), flush)
        rep = prefill_report(wl, Kp, ms, kern, peaks, peak_src)
        if Kp == cfg.k_pre[0]:
            rec["roofline"] = prefill_roofline(wl, Kp, kern, peaks, peak_src, rep["touched_experts"])
        rec["prefill"].append(rep)
    wl.status_ok("prefill")
    for M in cfg.pool_m:
        ms = wl.timed(lambda: wl.decode(M), steps, warmup, flush)
        kern = wl.kernel_times(lambda: wl.decode(M), min(steps, 6), flush)
        sp, keep = static_pool_for(wl, M)
        st = wl.timed(lambda: ex.exfold_moe_decode_static(wl.layer, wl.xd, wl.lgd, wl.wg, wl.wu, wl.wd, sp, wl.yd,
                                                          wl.ws), steps, warmup, flush)
        wl.decode(M)  # pool_size / yd of the dynamic pool again
        torch.cuda.synchronize()
        rep = decode_report(wl, M, ms, kern, peaks, static_ms=st)
        rl = decode_roofline(wl, kern, peaks, rep["effective_pool"])
        if rl:
            rep["roofline"] = rl
        rec["decode"].append(rep)
    wl.status_ok("decode")
    Kp0, M0 = cfg.k_pre[0], cfg.pool_m[0]
    if with_e2e:
        rec["e2e"] = e2e_leg(wl, Kp0, M0, min(steps, 6), flush)
    if with_cpu and not args.skip_cpu_baseline:
        wl.prefill(Kp0)
        wl.decode(M0)
        torch.cuda.synchronize()
        rec["cpu_baseline"], rec["parity_sample"] = cpu_baseline_leg(wl, Kp0, M0, args.cpu_flop_budget)
    if stack_layers:
        rec["stack"] = [stack_leg(wl, M0, stack_layers, flush), stack_leg(wl, M0, stack_layers, flush, Kp=Kp0)]
    if sweep:
        rec["decode_sweep"] = decode_sweep(wl, sweep[0], sweep[1], peaks, flush, max(4, steps // 2), warmup)
    wl.free()
    return rec


def decode_sweep(wl, batches, pools, peaks, flush, steps, warmup):
    """Decode batch x pool sweep: us/layer, effective pool, GB/s on the pool's weight bytes, speed-up over the
    unfolded layer (M = N) of the same batch."""
    cfg = wl.cfg
    N, K = cfg.n_experts, cfg.top_k
    table = []
    for B in [b for b in batches if b * K <= 4096]:
        wl.set_batch(B)
        row = {}
        for M in pools:
            ms = wl.timed(lambda: wl.decode(M), steps, warmup, flush)
            row[M] = decode_report(wl, M, ms, None, peaks)
        for M in pools:
            r = row[M]
            table.append({"B": B, "M": M, "P": r["effective_pool"], "us": r["us_per_layer"],
                          "gbs": r["gbs_on_pool_bytes"], "frac_hbm": r["frac_of_measured_hbm"],
                          "speedup_vs_unfolded": r4(row[N]["us_per_layer"] / r["us_per_layer"])})
    wl.status_ok("the decode sweep")
    return table


def describe(cfg):
    return (f"{cfg.name}-shaped layer: N={cfg.n_experts}+{cfg.n_shared} experts, d={cfg.hidden}, I={cfg.inter}, "
            f"top-{cfg.top_k} folded to top-{'/'.join(map(str, cfg.k_pre))}, prefill T={cfg.prefill_tokens}; decode "
            f"B={cfg.decode_batch}, pool M={'/'.join(map(str, cfg.pool_m))}; logits {cfg.logits}")


def run_ours(args, rank, world):
    import torch
    import torch.distributed as dist
    from paper_2608_24938_b200 import binding as ex

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    cfg = workload_config(args)
    Kp = args.k_pre or cfg.k_pre[0]
    M = args.pool_m or cfg.pool_m[0]
    K, N, d, I = cfg.top_k, cfg.n_experts, cfg.hidden, cfg.inter
    peaks, peak_src = load_peaks()
    warmup = max(args.warmup, 3)
    wl = Workload(ex, cfg, dev)
    T, B = wl.T, wl.B
    flush = Flush(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        flush()
        wl.prefill(Kp)
        wl.decode(M)
    torch.cuda.synchronize()
    wl.status_ok("warm-up")
    pool_size = int(wl.dmeta["pool_size"].item())

    # ---- timed region: K steps, per-call CUDA events on the launching stream, L2 flushed between calls
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    launches0 = ex.exfold_launch_count()
    wall0 = time.perf_counter()
    for k in range(args.steps):
        flush()
        ev[k][0].record()
        wl.prefill(Kp)
        ev[k][1].record()
        flush()
        ev[k][2].record()
        wl.decode(M)
        ev[k][3].record()
    barrier()
    wall = time.perf_counter() - wall0
    launches = ex.exfold_launch_count() - launches0
    clocks = sampler.finish()
    wl.status_ok("the timed region")
    pre_list = [e[0].elapsed_time(e[1]) for e in ev]
    dec_list = [e[2].elapsed_time(e[3]) for e in ev]
    pre_ms, dec_ms = max_over_ranks([float(np.mean(pre_list)), float(np.mean(dec_list))], world, dev)
    pre_list = [v * pre_ms / float(np.mean(pre_list)) for v in pre_list]  # scaled to the slowest rank's mean
    dec_list = [v * dec_ms / float(np.mean(dec_list)) for v in dec_list]

    # ---- per-kernel durations (CUDA events recorded by the library around each launch)
    nprof = min(args.steps, 10)
    kern_p = wl.kernel_times(lambda: wl.prefill(Kp), nprof, flush)
    kern_d = wl.kernel_times(lambda: wl.decode(M), nprof, flush)
    pre_rep = prefill_report(wl, Kp, pre_list, kern_p, peaks, peak_src, world)
    wl.decode(M)
    torch.cuda.synchronize()
    dec_rep = decode_report(wl, M, dec_list, kern_d, peaks)
    rl_d = decode_roofline(wl, kern_d, peaks, pool_size)
    if rl_d:
        dec_rep["roofline"] = rl_d
    if world == 1:
        sp, keep = static_pool_for(wl, M)
        st = wl.timed(lambda: ex.exfold_moe_decode_static(wl.layer, wl.xd, wl.lgd, wl.wg, wl.wu, wl.wd, sp, wl.yd,
                                                          wl.ws), min(args.steps, 10), 3, flush)
        dec_rep["static_pool_us_per_layer"] = r4(float(np.mean(st)) * 1e3)

    # ---- sustained leg: the headline prefill call back to back for >= 2 s (inputs far exceed L2: no flush needed)
    sustained = None
    if not args.skip_sustained:
        n_calls = int(max(10, min(20000, 2.2e3 / pre_ms)))
        s2 = ClockSampler(local, period=0.01)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s2.start()
        e0.record()
        for _ in range(n_calls):
            wl.prefill(Kp)
        e1.record()
        barrier()
        ck = s2.finish()
        sus_ms = max_over_ranks([e0.elapsed_time(e1) / n_calls], world, dev)[0]
        tf = pre_rep["flop"] / (sus_ms * 1e-3) / 1e12
        sustained = {"calls": n_calls, "seconds": r4(sus_ms * n_calls * 1e-3), "ms_per_call": r4(sus_ms),
                     "useful_tflops": r4(tf), "frac_of_bf16_sustained": r4(tf / peaks["bf16_tflops_sustained"]),
                     "frac_of_bf16_peak": r4(tf / peaks["bf16_tflops"]), "clocks": ck}
        wl.status_ok("the sustained leg")

    # ---- end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
    e2e = e2e_leg(wl, Kp, M, min(args.steps, 10), flush, world)

    out = {
        "metric": "folded-MoE-layer prefill tokens/s (decode us/layer and roofline fractions alongside)",
        "value": job_tokens_per_s(T, world, pre_ms),
        "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": pre_ms + dec_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": f"{cfg.name}-shaped layer: N={N}+{cfg.n_shared} experts, d={d}, I={I}, top-{K} folded to "
                               f"top-{Kp}, prefill T={T}; decode B={B}, pool M={M} (effective {pool_size})",
                   "replicas": world, "l2": "512 MiB buffer read between calls (L2 evicted, lines clean); weights also exceed L2",
                   "logits": cfg.logits, "seed": cfg.seed},
        "prefill": pre_rep,
        "decode": dec_rep,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": e2e,
        "peaks": {"source": peak_src, **peaks, "nominal": NOMINAL},
        "wall_s_timed_region": r4(wall),
    }
    if sustained:
        out["sustained"] = sustained
    rl = prefill_roofline(wl, Kp, kern_p, peaks, peak_src, pre_rep["touched_experts"])
    if rl:
        out["roofline"] = rl
    if args.layers > 0 and world == 1:
        out["stack"] = [stack_leg(wl, M, args.layers, flush), stack_leg(wl, M, args.layers, flush, Kp=Kp)]

    # ---- CPU baseline: the oracle as it stands, bounded sample, rank 0 at N=1
    if rank == 0 and world == 1 and not args.skip_cpu_baseline:
        wl.prefill(Kp)
        wl.decode(M)
        torch.cuda.synchronize()
        out["cpu_baseline"], out["parity_sample"] = cpu_baseline_leg(wl, Kp, M, args.cpu_flop_budget)

    # ---- every other benchmark configuration (one GPU, whole-suite run only)
    if world == 1 and rank == 0 and not args.workload and not args.skip_configs:
        wl.free()
        steps_c = min(args.steps, 12)
        out["configs"] = {}
        t0 = time.time()
        for name in ("mixtral", "qwen3", "tiny"):
            sweep = ((1, 8, 32, 128, 256), (8, 16, 32, 64, 128)) if name == "qwen3" else None
            out["configs"][name] = measure_config(ex, si.CONFIGS[name], dev, args, peaks, peak_src, flush, steps_c, 3,
                                                  sweep=sweep, stack_layers=args.layers if name == "qwen3" else 0)
            log(f"[bench] config {name} done at +{time.time() - t0:.0f}s")
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_decode_sweep(args):
    """Decode batch x pool sweep on one workload's layer (default: the Qwen3-shaped one). One GPU, one JSON line."""
    import torch
    from paper_2608_24938_b200 import binding as ex

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = si.CONFIGS[args.workload or "qwen3"]
    peaks, peak_src = load_peaks()
    batches = (1, 8, 32, 128, 256)
    pools = sorted({m for m in (8, 16, 32, 64, 128) if m < cfg.n_experts} | {cfg.n_experts})
    wl = Workload(ex, si.scaled(cfg, prefill_tokens=8), dev, batches=batches)
    table = decode_sweep(wl, batches, pools, peaks, Flush(dev), args.steps, max(args.warmup, 3))
    print(json.dumps({"metric": "decode sweep: us/layer and GB/s on pool weight bytes", "workload": cfg.name,
                      "unit": "us/layer", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
                      "dtype": cfg.dtype, "data": "synthetic", "peaks": {"source": peak_src, **peaks},
                      "l2": "512 MiB buffer read between calls", "table": table}), flush=True)


def run_reference(args, rank, world):
    """The reference arm of this benchmark is the CPU oracle (the paper ships no code to install)."""
    if rank != 0:
        return
    import oracle
    cfg = workload_config(args)
    Kp = args.k_pre or cfg.k_pre[0]
    M = args.pool_m or cfg.pool_m[0]
    T, B, K, N, d, I = cfg.prefill_tokens, cfg.decode_batch, cfg.top_k, cfg.n_experts, cfg.hidden, cfg.inter
    inp = build_inputs(cfg, T, B)
    probe = oracle_sample_run(cfg, inp, Kp, max(2, oracle.num_threads()))
    per_tok = probe["seconds"] / probe["tokens"]
    budget = 150.0 / (args.steps + args.warmup)
    n_s = int(max(1, min(T, 1024, budget / per_tok)))
    times = []
    for it in range(args.warmup + args.steps):
        r = oracle_sample_run(cfg, inp, Kp, n_s, seed=100 + it)
        if it >= args.warmup:
            times.append(r["seconds"])
    sec = float(np.mean(times))
    val = n_s / sec
    sample = f"each step: {n_s} seeded prefill tokens (all their routes), routing at full size"
    out = {"impl": "reference",
           "metric": "folded-MoE-layer prefill tokens/s (decode us/layer and roofline fractions alongside)",
           "value": val, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": cfg.dtype, "data": "synthetic",
           "config": {"workload": f"{cfg.name}-shaped layer: N={N}+{cfg.n_shared} experts, d={d}, I={I}, top-{K} "
                                  f"folded to top-{Kp}, prefill T={T}; decode B={B}, pool M={M}", "sample": sample},
           "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(si.CONFIGS),
                    help="measure only this layer (default: the GLM-4.5-Air-shaped headline plus every other config)")
    ap.add_argument("--k-pre", type=int, default=0)
    ap.add_argument("--pool-m", type=int, default=0)
    ap.add_argument("--tokens", type=int, default=0, help="override the prefill token count (reduced cases for profiling)")
    ap.add_argument("--batch", type=int, default=0, help="override the decode batch")
    ap.add_argument("--inter", type=int, default=0, help="override the expert intermediate size")
    ap.add_argument("--experts", type=int, default=0, help="override the number of routed experts")
    ap.add_argument("--layers", type=int, default=4,
                    help="also time stacks of this many layers (router scores + folded layer each, decode and prefill), "
                         "launched on the stream and replayed as one CUDA graph (0: skip)")
    ap.add_argument("--decode-sweep", action="store_true",
                    help="instead of the benchmark line: decode batch x pool sweep on --workload (one GPU)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-sustained", action="store_true")
    ap.add_argument("--skip-configs", action="store_true")
    ap.add_argument("--cpu-flop-budget", type=float, default=3e12,
                    help="flop of oracle work in the cpu-baseline sample (about 10-30 s of CPU time)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.decode_sweep:
        if rank == 0:
            run_decode_sweep(args)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world)


if __name__ == "__main__":
    main()
