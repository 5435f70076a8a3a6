"""CPU oracle for the folded MoE layer: test infrastructure, never on the product path.

Thin ctypes wrappers around exfold_oracle.c (plain C, double arithmetic, written
from the paper's equations). Only tests, the smoke check and the benchmark's
cpu-baseline leg may import this package.
"""
from .oracle import (build, calibrate, decode_eq4, decode_fold, decode_static, expert_outputs, gate, moe_apply,
                     num_threads, prefill_eq4, prefill_fold, prefill_fold_safe, router_logits, sort_routes,
                     static_pool)

__all__ = ["build", "calibrate", "decode_eq4", "decode_fold", "decode_static", "expert_outputs", "gate",
           "moe_apply", "num_threads", "prefill_eq4", "prefill_fold", "prefill_fold_safe", "router_logits", "sort_routes",
           "static_pool"]
