"""Writes tests/golden/oracle_tiny.json: a regression snapshot of the CPU oracle on the tiny seeded layer.

It calls only the oracle (and the seeded input generator); nothing here comes from the CUDA path.
Run from the repository root:  python tests/golden/make_oracle_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402
import synth_inputs as si  # noqa: E402


def snapshot():
    cfg = si.CONFIGS["tiny"]
    A = si.as_oracle_array
    x, lg = si.hidden_states(cfg, cfg.prefill_tokens), si.router_logits(cfg, cfg.prefill_tokens)
    xd, lgd = si.hidden_states(cfg, cfg.decode_batch, "x_dec"), si.router_logits(cfg, cfg.decode_batch, "logits_dec")
    wg, wu, wd = si.expert_weights(cfg, std=0.02, correlated=0.8)
    xc, lc = si.hidden_states(cfg, cfg.calib_tokens, "x_cal"), si.router_logits(cfg, cfg.calib_tokens, "logits_cal")
    cal = oracle.calibrate(A(xc), lc.numpy(), A(wg), A(wu), A(wd), cfg.n_experts, cfg.top_k)
    pre = oracle.prefill_fold(lg.numpy(), cfg.top_k, 1, cal["S"], cal["L"], cal["h"], cal["lnh"])
    y = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), pre["ids"], pre["w"], cfg.n_experts)
    dec = oracle.decode_fold(lgd.numpy(), cfg.top_k, 4, cal["S"], cal["L"], cal["h"])
    yd = oracle.moe_apply(A(xd), A(wg), A(wu), A(wd), dec["ids"], dec["w"], cfg.n_experts)
    return {
        "config": "tiny (N=8, d=128, I=256, top-2 -> top-1, decode B=16 M=4), correlated experts rho=0.8, seed %d" % cfg.seed,
        "S_row0": [float(v) for v in cal["S"][0]],
        "L_row0": [float(v) for v in cal["L"][0]],
        "h": [float(v) for v in cal["h"]],
        "prefill_ids_first16": pre["ids"][:16, 0].tolist(),
        "prefill_w_first8": [float(v) for v in pre["w"][:8, 0]],
        "prefill_y_norm": float(np.linalg.norm(y.astype(np.float64))),
        "prefill_y_first4": [float(v) for v in y[0, :4]],
        "decode_pool": dec["pool_ids"].tolist(),
        "decode_ids_first8": dec["ids"][:8].reshape(-1).tolist(),
        "decode_y_norm": float(np.linalg.norm(yd.astype(np.float64))),
    }


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_tiny.json")
    with open(out, "w") as f:
        json.dump(snapshot(), f, indent=1)
    print("wrote", out)
