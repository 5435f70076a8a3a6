"""Per-k-block timing of the prefill grouped GEMM's MMA thread (a development tool, not part of the layer).

Builds a trace variant of the library (-DEXFOLD_TRACE: one CTA logs the cycle counter and the ns timer each time a
k-block's operands are ready), runs one Mixtral-/Qwen3-/GLM-shaped prefill call and prints the distribution of the
intervals between consecutive k-blocks. A k-block is four M128 N256 K16 MMAs: 512 cycles at the nominal rate.

    python -m paper_2608_24938_b200.kblock_trace --workload mixtral --gemm 1
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
    args = ap.parse_args()
    tmp = tempfile.mkdtemp(prefix="exfold_trace_")
    lib = b.build(force=True, extra_flags=("-DEXFOLD_TRACE", "-rdc=true", f"-DEXFOLD_TRACE_KB_MODE={args.gemm - 1}"),
                  lib_path=os.path.join(tmp, "libexfold_trace.so"), obj_dir=os.path.join(tmp, "obj"))
    ex = load_binding(lib)
    ex.lib.exfold_debug_read_trace.restype = C.c_int
    ex.lib.exfold_debug_read_trace.argtypes = [C.c_void_p]
    cfg = si.CONFIGS[args.workload]
    dev = torch.device("cuda:0")
    T, K, N, d, I = cfg.prefill_tokens, cfg.top_k, cfg.n_experts, cfg.hidden, cfg.inter
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
    flat = buf[3].reshape(-1).astype(np.int64)
    cyc, ns = flat[:KB], flat[KB:2 * KB]
    n = int((cyc > 0).sum())
    cyc, ns = cyc[:n], ns[:n]
    dc = np.diff(cyc)
    per_tile = (d if args.gemm == 1 else I) // 64
    print(f"{args.workload} GEMM-{args.gemm}: {n} k-blocks of one CTA, {per_tile} per tile; "
          f"SM clock inside the kernel {(cyc[-1] - cyc[0]) / (ns[-1] - ns[0]):.3f} GHz")
    print(f"cycles between k-blocks: median {np.median(dc):.0f}, mean {dc.mean():.0f}, p90 {np.percentile(dc, 90):.0f}, "
          f"max {dc.max()}  (four MMAs at the nominal rate: 512)")
    edges = [0, 520, 640, 800, 1000, 1500, 2500, 5000, 10 ** 9]
    hist, _ = np.histogram(dc, bins=edges)
    print("histogram:", ", ".join(f">={e}: {h}" for e, h in zip(edges[:-1], hist.tolist())))


if __name__ == "__main__":
    main()
