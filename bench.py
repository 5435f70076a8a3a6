#!/usr/bin/env python
"""Benchmark of the folded-MoE layer (ExFold hot path) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mixtral|qwen3|glm45air|tiny]
                    [--k-pre K'] [--pool-m M] [--impl ours|reference]

One step = one pass of the whole hot path: a prefill call over T tokens (token-level Top-K'
folding) followed by a decode call over a batch of B tokens (pool-M folding), on seeded
synthetic inputs shaped like the named model. Prints ONE JSON line (rank 0):
  value        prefill tokens/s of the whole job, inputs resident in HBM (device-timed, max over ranks)
  decode       microseconds per decode layer and its HBM roofline
  e2e          the same metric through the host-buffer entry points (pinned host x/logits in, y out)
  roofline     dominant prefill kernel (grouped GEMM-1) against the measured bf16 tensor peak
  cpu_baseline the CPU oracle timed on this machine's host cores on a bounded sample (rank 0, N=1)
With N > 1 (torchrun) every rank runs an independent replica of the layer: the path has no
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

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes measured by ncu (dram__bytes_read.sum + dram__bytes_write.sum) divided by the algorithmic
# bytes of the same launch, from the reduced-case ncu captures whose summaries are under profiles/.
# Traffic grows with the weights, so the full-size figure is this ratio times the full-size algorithmic bytes.
NCU_TRAFFIC_RATIO = {"gemm1": 511.3 / 502.3, "decode_gateup": 239.3 / 234.9}


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
    log(f"[bench] inputs generated in {time.time() - t0:.1f}s")
    return inp


def oracle_sample_run(cfg, inp, Kp, M, n_tokens, seed=7):
    """CPU oracle on a seeded sample of prefill tokens (routing at full size) and on the full decode batch."""
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


def workload_config(args):
    cfg = si.CONFIGS[args.workload]
    over = {}
    if args.tokens:
        over["prefill_tokens"] = args.tokens
    if args.batch:
        over["decode_batch"] = args.batch
    if args.inter:
        over["inter"] = args.inter
    if over:
        cfg = si.scaled(cfg, name=cfg.name + "-reduced", **over)
    return cfg


def stack_leg(ex, cfg, layer, tables, weights, xd, M, L, dev, flush, reps=10):
    """L decode layers of the workload's shape, each = router scores (W_r x) + folded decode layer, one after the
    other on one stream. Every layer owns its weights (device copies rolled along the expert axis, so no weight
    line is reused between layers) and its router matrix; all layers read the same x (the layers are sequential
    in time, independent in data). Timed as plain stream launches and as one captured CUDA graph."""
    import torch
    wg, wu, wd = weights
    B, N, d = xd.shape[0], cfg.n_experts, cfg.hidden
    per = [(torch.roll(wg, l, 0), torch.roll(wu, l, 0), torch.roll(wd, l, 0)) if l else (wg, wu, wd) for l in range(L)]
    wr0 = si.router_weights(cfg).to(dev)
    wrs = [torch.roll(wr0, l, 0) for l in range(L)]
    lgs = [torch.empty((B, N), dtype=torch.float32, device=dev) for _ in range(L)]
    ys = [torch.empty((B, d), dtype=wg.dtype, device=dev) for _ in range(L)]
    ws = ex.alloc_workspace(layer, B, cfg.top_k)

    def run_layers():
        for l in range(L):
            ex.exfold_router_logits(layer, xd, wrs[l], lgs[l], ws)
            ex.exfold_moe_decode(layer, xd, lgs[l], per[l][0], per[l][1], per[l][2], tables, M, ys[l], ws)

    def timed(fn):
        ts = []
        for it in range(reps + 2):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    res = {"layers": L, "what": "router GEMM + folded decode layer per layer, own weights per layer, same x"}
    res["stream_us_per_layer"] = timed(run_layers) * 1e3 / L
    assert ex.exfold_device_status(ws) == 0, "device status after the layer stack"
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            run_layers()
        torch.cuda.synchronize()
        res["graph_us_per_layer"] = timed(graph.replay) * 1e3 / L
        assert ex.exfold_device_status(ws) == 0, "device status after the graph replays"
    except Exception as e:  # capture is an optional measurement: report, do not lose the benchmark line
        res["graph_error"] = f"{type(e).__name__}: {e}"[:300]
    return res


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
    T, B, K, N, d, I = cfg.prefill_tokens, cfg.decode_batch, cfg.top_k, cfg.n_experts, cfg.hidden, cfg.inter
    peaks, peak_src = load_peaks()
    inp = build_inputs(cfg, T, B)
    g = lambda t: t.to(dev)
    x, lg, xd, lgd = g(inp["x"]), g(inp["lg"]), g(inp["xd"]), g(inp["lgd"])
    wg, wu, wd = g(inp["wg"]), g(inp["wu"]), g(inp["wd"])
    tabs = [g(t) for t in inp["tables"]]
    tables = ex.make_tables(*tabs)
    layer = ex.make_layer(N, cfg.n_shared, d, I, K, cfg.dtype)
    ws = ex.alloc_workspace(layer, max(T, B), max(Kp, K), host_staging=True)
    y = torch.empty((T, d), dtype=wg.dtype, device=dev)
    yd = torch.empty((B, d), dtype=wg.dtype, device=dev)
    dmeta = dict(pool_size=torch.zeros(1, dtype=torch.int32, device=dev))
    flush_buf = torch.zeros(128 << 20, dtype=torch.int32, device=dev)  # 512 MiB, > 4x L2

    class _Flush:
        """Evicts L2 between calls by READING a 512 MiB buffer: the cache is left full of clean lines.
        (Writing the buffer instead would leave ~126 MB of dirty lines whose write-back is then charged to
        the first reads of the timed kernel: about 20 us of foreign DRAM traffic per call.)"""

        def zero_(self):
            torch.sum(flush_buf)

    flush = _Flush()

    def prefill():
        ex.exfold_moe_prefill(layer, x, lg, wg, wu, wd, tables, Kp, y, ws)

    def decode():
        ex.exfold_moe_decode(layer, xd, lgd, wg, wu, wd, tables, M, yd, ws, meta=dmeta)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        prefill()
        decode()
    torch.cuda.synchronize()
    assert ex.exfold_device_status(ws) == 0, "device status after warm-up"
    pool_size = int(dmeta["pool_size"].item())

    # ---- timed region: K steps, per-call CUDA events on the launching stream, L2 flushed between calls
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    launches0 = ex.exfold_launch_count()
    wall0 = time.perf_counter()
    for k in range(args.steps):
        flush.zero_()
        ev[k][0].record()
        prefill()
        ev[k][1].record()
        flush.zero_()
        ev[k][2].record()
        decode()
        ev[k][3].record()
    barrier()
    wall = time.perf_counter() - wall0
    launches = ex.exfold_launch_count() - launches0
    sampler.stop_flag.set()
    sampler.join()
    assert ex.exfold_device_status(ws) == 0, "device status after the timed region"
    pre_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    dec_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in ev]))
    pre_min = float(np.min([e[0].elapsed_time(e[1]) for e in ev]))
    dec_min = float(np.min([e[2].elapsed_time(e[3]) for e in ev]))
    pre_ms, dec_ms = max_over_ranks([pre_ms, dec_ms], world, dev)

    # ---- per-kernel durations (CUDA events recorded by the library around each launch)
    ex.exfold_profile_enable(True)
    kern = {}
    nprof = min(args.steps, 10)
    for _ in range(nprof):
        flush.zero_()
        prefill()
        torch.cuda.synchronize()
        for k_, v in ex.exfold_profile_read().items():
            kern.setdefault(k_, []).append(v)
        flush.zero_()
        decode()
        torch.cuda.synchronize()
        for k_, v in ex.exfold_profile_read().items():
            kern.setdefault("dec:" + k_ if k_ == "convert_bf16" else k_, []).append(v)
    ex.exfold_profile_enable(False)
    kern = {k_: float(np.mean(v)) for k_, v in kern.items()}

    # ---- end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
    xh, lh = inp["x"].pin_memory(), inp["lg"].pin_memory()
    xdh, ldh = inp["xd"].pin_memory(), inp["lgd"].pin_memory()
    yh = torch.empty((T, d), dtype=wg.dtype).pin_memory()
    ydh = torch.empty((B, d), dtype=wg.dtype).pin_memory()
    ne2e = min(args.steps, 10)
    ee = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(ne2e)]
    for it in range(ne2e + 2):
        k = max(it - 2, 0)
        flush.zero_()
        ee[k][0].record()
        ex.exfold_moe_prefill_host(layer, xh, lh, wg, wu, wd, tables, Kp, yh, ws)
        ee[k][1].record()
        flush.zero_()
        ee[k][2].record()
        ex.exfold_moe_decode_host(layer, xdh, ldh, wg, wu, wd, tables, M, ydh, ws)
        ee[k][3].record()
        torch.cuda.synchronize()
    e2e_pre = float(np.mean([e[0].elapsed_time(e[1]) for e in ee]))
    e2e_dec = float(np.mean([e[2].elapsed_time(e[3]) for e in ee]))
    e2e_pre, e2e_dec = max_over_ranks([e2e_pre, e2e_dec], world, dev)
    el = 2 if cfg.dtype == "bf16" else 4
    h2d = T * d * el + T * N * 4 + B * d * el + B * N * 4
    d2h = T * d * el + B * d * el

    # ---- optional: a stack of decode layers (router GEMM + folded decode layer), stream launches vs one CUDA graph
    stack = None
    if args.layers > 0 and world == 1:
        stack = stack_leg(ex, cfg, layer, tables, (wg, wu, wd), xd, M, args.layers, dev, flush)

    # ---- algorithmic work
    rows = T * Kp + T * cfg.n_shared
    flop_layer = rows * 6.0 * d * I
    flop_gemm1 = rows * 4.0 * d * I
    pool_bytes = (pool_size + cfg.n_shared) * 3.0 * d * I * el
    gateup_bytes = pool_bytes * 2.0 / 3.0
    out = {
        "metric": "folded-MoE-layer prefill tokens/s (decode us/layer and roofline fractions alongside)",
        "value": job_tokens_per_s(T, world, pre_ms),
        "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": pre_ms + dec_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": f"{cfg.name}-shaped layer: N={N}+{cfg.n_shared} experts, d={d}, I={I}, top-{K} folded to "
                               f"top-{Kp}, prefill T={T}; decode B={B}, pool M={M} (effective {pool_size})",
                   "replicas": world, "l2": "512 MiB buffer read between calls (L2 evicted, lines clean); weights also exceed L2",
                   "logits": cfg.logits, "seed": cfg.seed},
        "prefill": {"ms": pre_ms, "ms_min": pre_min, "tokens_per_s_per_gpu": T / (pre_ms * 1e-3),
                    "useful_tflops": flop_layer / (pre_ms * 1e-3) / 1e12,
                    "frac_of_bf16_peak": flop_layer / (pre_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "frac_of_bf16_sustained": flop_layer / (pre_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]},
        "decode": {"us_per_layer": dec_ms * 1e3, "us_min": dec_min * 1e3, "pool_weight_bytes": pool_bytes,
                   "layer_gbs": pool_bytes / (dec_ms * 1e-3) / 1e9,
                   "layer_frac_of_hbm": pool_bytes / (dec_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "kernels_ms": kern,
        "gpu_launches": int(launches),
        "clocks": sampler.summary(),
        "e2e": {"value": job_tokens_per_s(T, world, e2e_pre), "unit": "tokens/s", "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "prefill_ms": e2e_pre, "decode_us": e2e_dec * 1e3},
        "peaks": {"source": peak_src, **peaks},
        "wall_s_timed_region": wall,
    }
    if stack is not None:
        out["stack"] = stack
    if "gemm1_gateup_swiglu" in kern:
        t1 = kern["gemm1_gateup_swiglu"] * 1e-3
        ach = flop_gemm1 / t1 / 1e12
        touched = N + cfg.n_shared  # every expert receives rows at these sizes
        bytes_gemm1 = touched * 2.0 * d * I * el + rows * d * el + rows * I * el
        out["roofline"] = {"kernel": "grouped GEMM-1 (gate/up + SwiGLU), tcgen05", "bound": "tensor", "achieved": ach,
                           "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
                           "traffic": bytes_gemm1 * NCU_TRAFFIC_RATIO["gemm1"],
                           "traffic_note": "ncu reduced-case DRAM bytes / algorithmic bytes x full-size algorithmic bytes",
                           "peak_source": f"{peak_src} burst bf16 matmul",
                           "launch_ms": kern["gemm1_gateup_swiglu"], "flop_per_launch": flop_gemm1}
    elif "simt_ffn" in kern:
        t1 = kern["simt_ffn"] * 1e-3
        ach = flop_layer / t1 / 1e12
        out["roofline"] = {"kernel": "SIMT fp32 expert FFN", "bound": "alu", "achieved": ach, "peak": 72.0,
                           "unit": "TFLOP/s", "frac": ach / 72.0, "traffic": None,
                           "peak_source": "148 SMs x 128 fp32 lanes x 2 x 1.9 GHz"}
    if "decode_gateup" in kern:
        tg = kern["decode_gateup"] * 1e-3
        td = kern.get("decode_down", 0.0) * 1e-3
        out["decode"]["roofline"] = {"kernel": "decode GEMM-1 (gate/up weight stream over the pool), tcgen05", "bound": "hbm",
                                     "achieved": gateup_bytes / tg / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                     "frac": gateup_bytes / tg / 1e9 / peaks["hbm_gbs"],
                                     "traffic": gateup_bytes * NCU_TRAFFIC_RATIO["decode_gateup"],
                                     "bytes_per_launch": gateup_bytes, "launch_ms": kern["decode_gateup"]}
        if td > 0:
            out["decode"]["down_gbs"] = pool_bytes / 3.0 / td / 1e9
            out["decode"]["ffn_gbs"] = pool_bytes / (tg + td) / 1e9

    # ---- CPU baseline: the oracle as it stands, bounded sample, rank 0 at N=1
    if rank == 0 and world == 1 and not args.skip_cpu_baseline:
        import oracle
        per_tok = (Kp + cfg.n_shared) * 6.0 * d * I
        n_s = int(max(1, min(256, args.cpu_flop_budget / per_tok)))
        t0 = time.time()
        o = oracle_sample_run(cfg, inp, Kp, M, n_s)
        yg = y.float().cpu().numpy()[o["idx"]]
        emax, efro = rel_err(yg, o["y"])
        out["cpu_baseline"] = {"value": o["tokens_per_s"], "unit": "tokens/s", "cores": oracle.num_threads(),
                               "kind": "oracle",
                               "sample": f"{o['tokens']} seeded prefill tokens (all their routes) of the same "
                                         f"workload; routing at full size; {o['seconds']:.1f}s"}
        out["parity_sample"] = {"prefill_max_err_rel": emax, "prefill_fro_err_rel": efro, "tokens": int(o["tokens"])}
        if B * (K + cfg.n_shared) * 6.0 * d * I <= 4 * args.cpu_flop_budget:
            od = oracle_decode_run(cfg, inp, M)
            dmax, dfro = rel_err(yd.float().cpu().numpy(), od["y"])
            out["cpu_baseline"]["decode_us_per_layer"] = od["seconds"] * 1e6
            out["parity_sample"].update({"decode_max_err_rel": dmax, "decode_fro_err_rel": dfro})
        log(f"[bench] cpu baseline took {time.time() - t0:.1f}s")
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_decode_sweep(args):
    """Decode batch x pool sweep on one workload's layer (default: the Qwen3-shaped one): us/layer, effective pool,
    GB/s on the pool's weight bytes, speed-up over the unfolded layer (M = N). One GPU, one JSON line."""
    import torch
    from paper_2608_24938_b200 import binding as ex

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = si.CONFIGS[args.workload]
    peaks, peak_src = load_peaks()
    K, N, d, I = cfg.top_k, cfg.n_experts, cfg.hidden, cfg.inter
    batches = [b for b in (1, 8, 32, 128, 256) if b * K <= 4096]
    pools = sorted({m for m in (8, 16, 32, 64, 128) if m < N} | {N})
    inp = build_inputs(cfg, 8, max(batches))
    g = lambda t: t.to(dev)
    wg, wu, wd = g(inp["wg"]), g(inp["wu"]), g(inp["wd"])
    tables = ex.make_tables(*[g(t) for t in inp["tables"]])
    layer = ex.make_layer(N, cfg.n_shared, d, I, K, cfg.dtype)
    ws = ex.alloc_workspace(layer, max(batches), K)
    flush_buf = torch.zeros(128 << 20, dtype=torch.int32, device=dev)
    el = 2 if cfg.dtype == "bf16" else 4
    table = []
    for B in batches:
        xd, lgd = g(inp["xd"][:B].contiguous()), g(inp["lgd"][:B].contiguous())
        yd = torch.empty((B, d), dtype=wg.dtype, device=dev)
        meta = dict(pool_size=torch.zeros(1, dtype=torch.int32, device=dev))
        row = {}
        for M in pools:
            ts = []
            for it in range(args.steps + max(args.warmup, 3)):
                torch.sum(flush_buf)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                ex.exfold_moe_decode(layer, xd, lgd, wg, wu, wd, tables, M, yd, ws, meta=meta)
                e1.record()
                torch.cuda.synchronize()
                if it >= max(args.warmup, 3):
                    ts.append(e0.elapsed_time(e1))
            assert ex.exfold_device_status(ws) == 0
            us = float(np.mean(ts)) * 1e3
            pool = int(meta["pool_size"].item())
            byts = (pool + cfg.n_shared) * 3.0 * d * I * el
            row[M] = {"us": us, "pool": pool, "gbs": byts / (us * 1e-6) / 1e9}
        for M in pools:
            r = row[M]
            table.append({"B": B, "M": M, "effective_pool": r["pool"], "us_per_layer": round(r["us"], 2),
                          "gbs_on_pool_bytes": round(r["gbs"], 1),
                          "frac_of_measured_hbm": round(r["gbs"] / peaks["hbm_gbs"], 3),
                          "speedup_vs_unfolded": round(row[N]["us"] / r["us"], 3)})
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
    probe = oracle_sample_run(cfg, inp, Kp, M, max(2, oracle.num_threads()))
    per_tok = probe["seconds"] / probe["tokens"]
    budget = 150.0 / (args.steps + args.warmup)
    n_s = int(max(1, min(T, 1024, budget / per_tok)))
    times = []
    for it in range(args.warmup + args.steps):
        r = oracle_sample_run(cfg, inp, Kp, M, n_s, seed=100 + it)
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
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mixtral", choices=sorted(si.CONFIGS))
    ap.add_argument("--k-pre", type=int, default=0)
    ap.add_argument("--pool-m", type=int, default=0)
    ap.add_argument("--tokens", type=int, default=0, help="override the prefill token count (reduced cases for profiling)")
    ap.add_argument("--batch", type=int, default=0, help="override the decode batch")
    ap.add_argument("--inter", type=int, default=0, help="override the expert intermediate size")
    ap.add_argument("--layers", type=int, default=0,
                    help="also time a stack of this many decode layers (router scores + folded decode layer each), "
                         "launched on the stream and replayed as one CUDA graph")
    ap.add_argument("--decode-sweep", action="store_true",
                    help="instead of the benchmark line: decode batch x pool sweep on --workload (one GPU)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-flop-budget", type=float, default=3e11,
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
