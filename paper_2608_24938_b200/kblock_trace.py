"""Per-k-block timing of the prefill grouped GEMMs' MMA thread (a development tool, not part of the layer).

Builds a trace variant of the library (-DEXFOLD_TRACE: one CTA logs the cycle counter each time a k-block's operands
are ready, and the ns timer every 16th time), runs one prefill call and prints the distribution of the intervals
between consecutive k-blocks. A k-block is four K = 16 MMAs (M128 N256, or M256 N256 on a CTA pair): 512 cycles at
the tensor pipe's rate.

    python -m paper_2608_24938_b200.kblock_trace --workload mixtral --gemm 1
    python -m paper_2608_24938_b200.kblock_trace --workload glm45air --gemm 1 --pair --per-tile

--pair logs in the CTA-pair kernel (the leader of one pair) instead of the one-CTA kernel; --per-tile logs once per
work item instead of once per k-block (the logging itself costs ~50-70 cycles per k-block); --tokens overrides the
workload's prefill length.
"""
import argparse
import ctypes as C
import os
import sys
import tempfile
import types

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
import synth_inputs as si  # noqa: E402
from paper_2608_24938_b200 import build as b  # noqa: E402

KB = 1280


def load_binding(lib_path):
    """The package's ctypes binding, pointed at another build of the library."""
    path = os.path.join(ROOT, "paper_2608_24938_b200", "binding.py")
    src = open(path).read().replace('LIB_PATH = os.path.join(_HERE, "libexfold.so")', f"LIB_PATH = {lib_path!r}")
    mod = types.ModuleType("exfold_trace_binding")
    mod.__file__ = path
    exec(compile(src, path, "exec"), mod.__dict__)
    return mod


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="mixtral", choices=sorted(si.CONFIGS))
    ap.add_argument("--gemm", type=int, default=1, choices=[1, 2])
    ap.add_argument("--pair", action="store_true")
    ap.add_argument("--per-tile", action="store_true")
    ap.add_argument("--tokens", type=int, default=0)
    args = ap.parse_args()
    tmp = tempfile.mkdtemp(prefix="exfold_trace_")
    flags = ["-DEXFOLD_TRACE", "-rdc=true", f"-DEXFOLD_TRACE_KB_MODE={args.gemm - 1}"]
    flags += ["-DEXFOLD_TRACE_PAIR"] if args.pair else []
    flags += ["-DEXFOLD_TRACE_TILE"] if args.per_tile else []
    lib = b.build(force=True, extra_flags=tuple(flags),
                  lib_path=os.path.join(tmp, "libexfold_trace.so"), obj_dir=os.path.join(tmp, "obj"))
    ex = load_binding(lib)
    ex.lib.exfold_debug_read_trace.restype = C.c_int
    ex.lib.exfold_debug_read_trace.argtypes = [C.c_void_p]
    cfg = si.CONFIGS[args.workload]
    dev = torch.device("cuda:0")
    T, K, N, d, I = args.tokens or cfg.prefill_tokens, cfg.top_k, cfg.n_experts, cfg.hidden, cfg.inter
    x, lg = si.hidden_states(cfg, T).to(dev), si.router_logits(cfg, T).to(dev)
    wg, wu, wd = [t.to(dev) for t in si.expert_weights(cfg)]
    tables = ex.make_tables(*[t.to(dev) for t in si.synthetic_tables(cfg)])
    layer = ex.make_layer(N, cfg.n_shared, d, I, K, cfg.dtype)
    ws = ex.alloc_workspace(layer, T, K)
    y = torch.empty((T, d), dtype=wg.dtype, device=dev)
    flush = torch.zeros(128 << 20, dtype=torch.int32, device=dev)
    for _ in range(4):
        torch.sum(flush)
        ex.exfold_moe_prefill(layer, x, lg, wg, wu, wd, tables, cfg.k_pre[0], y, ws)
        torch.cuda.synchronize()
    buf = np.zeros((4, 160, 16), np.uint64)
    assert ex.lib.exfold_debug_read_trace(buf.ctypes.data) == 0
    if args.pair:
        polls, ready = int(buf[args.gemm - 1][10][12]), int(buf[args.gemm - 1][10][13])
        print(f"the logging CTA issued {polls} k-blocks; the next stage's operands were already complete at {ready} of its polls")
    flat = buf[3].reshape(-1).astype(np.int64)
    cyc, ns = flat[:KB], flat[KB:2 * KB]
    n = int((cyc > 0).sum())
    if n < 18:
        print(f"only {n} entries logged (the chosen kernel did not run, or ran too few items on the logging CTA)")
        return
    cyc, ns = cyc[:n], ns[:n]
    dc = np.diff(cyc)
    last = ((n - 1) // 16) * 16  # the ns timer is logged with every 16th entry
    per_tile = (d if args.gemm == 1 else I) // 64
    unit = "work items" if args.per_tile else "k-blocks"
    print(f"{args.workload} GEMM-{args.gemm}{' (CTA-pair kernel)' if args.pair else ''}: {n} {unit} of one CTA, {per_tile} k-blocks "
          f"per item; SM clock inside the kernel {(cyc[last] - cyc[0]) / max(1, ns[last] - ns[0]):.3f} GHz")
    scale = per_tile if args.per_tile else 1
    print(f"cycles per k-block: median {np.median(dc) / scale:.0f}, mean {dc.mean() / scale:.0f}, "
          f"p10 {np.percentile(dc, 10) / scale:.0f}, p90 {np.percentile(dc, 90) / scale:.0f}, max {dc.max() / scale:.0f}  "
          f"(four MMAs at the tensor pipe's rate: 512)")
    if args.per_tile:
        return
    edges = [0, 520, 640, 800, 1000, 1500, 2500, 5000, 10 ** 9]
    hist, _ = np.histogram(dc, bins=edges)
    print("histogram:", ", ".join(f">={e}: {h}" for e, h in zip(edges[:-1], hist.tolist())))


if __name__ == "__main__":
    main()
