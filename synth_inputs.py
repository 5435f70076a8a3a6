"""Seeded synthetic inputs for the folded-MoE layer.

This module only draws random tensors of the right shapes and distributions.
It contains none of the method's arithmetic (no routing, folding, calibration
or expert evaluation) and is the one piece shared by the CPU oracle's tests
and the CUDA path: both sides receive the very same host arrays.

Everything is generated on the host with numpy's Philox generator, one
independent sub-stream per (config seed, tensor tag, expert), so any tensor
can be regenerated alone and generation can run on several threads.
bf16 tensors are produced by rounding fp32 draws with torch (round to nearest
even) and are handed around as torch.bfloat16 CPU tensors.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor
from typing import Optional

import numpy as np
import torch

# tensor tags for the sub-streams
_TAG = {"x": 1, "logits": 2, "w_gate": 3, "w_up": 4, "w_down": 5, "tables": 6,
        "x_cal": 7, "logits_cal": 8, "zipf_perm": 9, "x_dec": 10, "logits_dec": 11,
        "corr_base": 12, "corr_gain": 13, "w_router": 14}


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    """One synthetic layer shaped like a model the paper evaluates (Appendix A, model table)."""
    name: str
    n_experts: int          # N routed experts
    n_shared: int           # 0 or 1 always-on shared expert (stored as expert index N)
    hidden: int             # d
    inter: int              # I
    top_k: int              # K
    dtype: str              # "f32" | "bf16"
    prefill_tokens: int     # T
    k_pre: tuple            # prefill budgets K'
    decode_batch: int       # B
    pool_m: tuple           # decode pool budgets M
    logits: str = "normal"  # "normal" | "zipf"
    zipf_s: float = 1.1
    seed: int = 20260824
    calib_tokens: int = 0   # >0: tables are really calibrated on this many tokens


CONFIGS = {
    # tiny fp32 layer: the oracle finishes it in well under a second
    "tiny": LayerConfig("tiny", 8, 0, 128, 256, 2, "f32", 64, (1,), 16, (4,), calib_tokens=512),
    # Mixtral-8x7B-shaped
    "mixtral": LayerConfig("mixtral", 8, 0, 4096, 14336, 2, "bf16", 4096, (1,), 32, (4,)),
    # Qwen3-30B-A3B-shaped, Zipf-skewed expert popularity
    "qwen3": LayerConfig("qwen3", 128, 0, 2048, 768, 8, "bf16", 8192, (4, 6), 64, (16, 32, 64),
                         logits="zipf"),
    # GLM-4.5-Air-shaped: 128 routed + 1 shared
    "glm45air": LayerConfig("glm45air", 128, 1, 4096, 1408, 8, "bf16", 16384, (4,), 128, (32,)),
}


def scaled(cfg: LayerConfig, **kw) -> LayerConfig:
    """A copy of cfg with some fields replaced (used for reduced parity cases)."""
    return dataclasses.replace(cfg, **kw)


def _rng(seed: int, tag: str, idx: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, _TAG[tag], idx])))


def _normal(seed: int, tag: str, idx: int, shape, std: float) -> np.ndarray:
    a = _rng(seed, tag, idx).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def to_dtype(a: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(a)
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def hidden_states(cfg: LayerConfig, n_tokens: int, tag: str = "x") -> torch.Tensor:
    """x ~ N(0,1), shape [n_tokens, d], in the layer dtype."""
    return to_dtype(_normal(cfg.seed, tag, 0, (n_tokens, cfg.hidden), 1.0), cfg.dtype)


def zipf_log_popularity(cfg: LayerConfig) -> np.ndarray:
    """ln p_sigma(e) with p_k proportional to k^-s over a seeded permutation of the experts."""
    n = cfg.n_experts
    p = np.arange(1, n + 1, dtype=np.float64) ** (-cfg.zipf_s)
    p /= p.sum()
    sigma = _rng(cfg.seed, "zipf_perm").permutation(n)
    out = np.empty(n, dtype=np.float64)
    out[sigma] = np.log(p)
    return out


def router_logits(cfg: LayerConfig, n_tokens: int, tag: str = "logits") -> torch.Tensor:
    """fp32 router logits [n_tokens, N]: N(0,1), plus ln(popularity) for the Zipf recipe."""
    z = _normal(cfg.seed, tag, 0, (n_tokens, cfg.n_experts), 1.0)
    if cfg.logits == "zipf":
        z = (z.astype(np.float64) + zipf_log_popularity(cfg)[None, :]).astype(np.float32)
    return torch.from_numpy(z)


def _one_expert(cfg: LayerConfig, tag: str, e: int, shape, std: float) -> torch.Tensor:
    return to_dtype(_normal(cfg.seed, tag, e, shape, std), cfg.dtype)


def router_weights(cfg: LayerConfig, std: Optional[float] = None) -> torch.Tensor:
    """Router matrix W_r [N, d] in the layer dtype, entries N(0, std); the default std = 1/sqrt(d) gives
    unit-variance scores on x ~ N(0, 1), like the logits generator's "normal" mode."""
    std = (1.0 / np.sqrt(cfg.hidden)) if std is None else std
    return to_dtype(_normal(cfg.seed, "w_router", 0, (cfg.n_experts, cfg.hidden), std), cfg.dtype)


def expert_weights(cfg: LayerConfig, std: float = 0.02, threads: Optional[int] = None,
                   correlated: float = 0.0):
    """(W_gate [E,I,d], W_up [E,I,d], W_down [E,d,I]) with E = N + n_shared, entries N(0, std).

    correlated = rho > 0 makes the down projections share a common component,
    W_down[e] = g_e (rho W_0 + sqrt(1-rho^2) W_e) with gains g_e spread over [1, 3.2],
    and gives all experts the same gate/up matrices, so that expert outputs are
    directionally aligned with different magnitudes (the geometry the paper's
    design-insight section describes).
    """
    E = cfg.n_experts + cfg.n_shared
    d, I = cfg.hidden, cfg.inter
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    wg = torch.empty((E, I, d), dtype=tdt)
    wu = torch.empty((E, I, d), dtype=tdt)
    wd = torch.empty((E, d, I), dtype=tdt)
    if correlated > 0.0:
        rho = float(correlated)
        base = _normal(cfg.seed, "corr_base", 0, (d, I), std)
        gains = np.exp(_rng(cfg.seed, "corr_gain").uniform(0.0, np.log(3.2), size=E))
        g0 = _normal(cfg.seed, "w_gate", 0, (I, d), std)
        u0 = _normal(cfg.seed, "w_up", 0, (I, d), std)
        for e in range(E):
            own = _normal(cfg.seed, "w_down", e, (d, I), std)
            wd[e] = to_dtype((gains[e] * (rho * base + np.sqrt(1 - rho * rho) * own)).astype(np.float32),
                             cfg.dtype)
            wg[e] = to_dtype(g0, cfg.dtype)
            wu[e] = to_dtype(u0, cfg.dtype)
        return wg, wu, wd

    def fill(job):
        tag, e = job
        if tag == "w_down":
            wd[e] = _one_expert(cfg, tag, e, (d, I), std)
        elif tag == "w_gate":
            wg[e] = _one_expert(cfg, tag, e, (I, d), std)
        else:
            wu[e] = _one_expert(cfg, tag, e, (I, d), std)

    jobs = [(t, e) for e in range(E) for t in ("w_gate", "w_up", "w_down")]
    nthr = threads or min(len(jobs), os.cpu_count() or 1)
    if nthr > 1 and E * d * I > (1 << 22):
        with ThreadPoolExecutor(nthr) as ex:
            list(ex.map(fill, jobs))
    else:
        for j in jobs:
            fill(j)
    return wg, wu, wd


def synthetic_tables(cfg: LayerConfig, unobserved_frac: float = 0.02):
    """Structured stand-in for calibrated tables (S, L, h, lnh), all fp32.

    h_e = exp(U(0, ln 3.2)) (norm spread of about 3x); a symmetric similarity
    c_st ~ U(0.2, 0.9); S_st = clip(c_st h_s / h_t, -4, 4); L_st = 1 - c_st^2;
    S_ee = 1, L_ee = 0; a seeded 2 % of the off-diagonal pairs is marked
    unobserved (S = 0, L = 1e30). A tenth of the observed off-diagonal scalars
    get a negative sign so that negative coefficients are exercised.
    """
    n = cfg.n_experts
    g = _rng(cfg.seed, "tables")
    h = np.exp(g.uniform(0.0, np.log(3.2), size=n))
    c = g.uniform(0.2, 0.9, size=(n, n))
    c = np.triu(c, 1)
    c = c + c.T
    S = np.clip(c * h[:, None] / h[None, :], -4.0, 4.0)
    neg = g.uniform(size=(n, n)) < 0.10
    S = np.where(neg, -S, S)
    L = 1.0 - c * c
    unob = g.uniform(size=(n, n)) < unobserved_frac
    S = np.where(unob, 0.0, S)
    L = np.where(unob, 1e30, L)
    np.fill_diagonal(S, 1.0)
    np.fill_diagonal(L, 0.0)
    h32 = h.astype(np.float32)
    lnh = np.log(h32.astype(np.float64)).astype(np.float32)
    return (torch.from_numpy(S.astype(np.float32)), torch.from_numpy(L.astype(np.float32)),
            torch.from_numpy(h32), torch.from_numpy(lnh))


def as_oracle_array(t: torch.Tensor) -> np.ndarray:
    """Host view handed to the oracle: fp32 arrays as they are, bf16 as raw uint16 bit patterns."""
    t = t.contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
