"""Shared helpers of the GPU parity tests: build a seeded case, run it through the C ABI,
run the oracle on the same host arrays, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import synth_inputs as si

A = si.as_oracle_array


class Case:
    """Host tensors of one layer + their device copies."""

    def __init__(self, cfg: si.LayerConfig, std: float = 0.05, correlated: float = 0.0, tables=None, T=None,
                 B=None):
        from paper_2608_24938_b200 import binding as ex
        self.ex = ex
        self.cfg = cfg
        self.dev = torch.device("cuda:0")
        self.T = T if T is not None else cfg.prefill_tokens
        self.B = B if B is not None else cfg.decode_batch
        self.x = si.hidden_states(cfg, self.T)
        self.lg = si.router_logits(cfg, self.T)
        self.xd = si.hidden_states(cfg, self.B, "x_dec")
        self.lgd = si.router_logits(cfg, self.B, "logits_dec")
        self.wg, self.wu, self.wd = si.expert_weights(cfg, std=std, correlated=correlated)
        self.tables_host = tables if tables is not None else si.synthetic_tables(cfg)
        self.layer = ex.make_layer(cfg.n_experts, cfg.n_shared, cfg.hidden, cfg.inter, cfg.top_k, cfg.dtype)
        g = lambda t: t.to(self.dev)
        self.d_x, self.d_lg, self.d_xd, self.d_lgd = g(self.x), g(self.lg), g(self.xd), g(self.lgd)
        self.d_wg, self.d_wu, self.d_wd = g(self.wg), g(self.wu), g(self.wd)
        self.set_tables(self.tables_host)
        self.ws = None

    def set_tables(self, tabs):
        self.tables_host = tuple(torch.as_tensor(t).contiguous() for t in tabs)
        self.d_tabs = [t.to(self.dev) for t in self.tables_host]
        self.tables = self.ex.make_tables(*self.d_tabs)

    def workspace(self, tokens, routes):
        need = self.ex.exfold_workspace_bytes(self.layer, tokens, routes)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(need, dtype=torch.uint8, device=self.dev)
        self.ws.fill_(0xFF)  # poison: anything the kernels forget to write shows up
        return self.ws

    def np_tables(self):
        return [t.numpy() for t in self.tables_host]

    # ---------------------------------------------------------------- GPU runs
    def run_prefill(self, Kp, with_meta=True, gemm_path=0):
        ex, cfg, T = self.ex, self.cfg, self.T
        K, N = cfg.top_k, cfg.n_experts
        ws = self.workspace(T, Kp)
        y = torch.full((T, cfg.hidden), float("nan"), dtype=self.d_wg.dtype, device=self.dev)
        meta = None
        if with_meta:
            i32 = dict(dtype=torch.int32, device=self.dev)
            meta = dict(ids=torch.full((T, Kp), -7, **i32),
                        w=torch.full((T, Kp), float("nan"), dtype=torch.float32, device=self.dev),
                        omit_src=torch.full((T, K - Kp), -7, **i32), omit_tgt=torch.full((T, K - Kp), -7, **i32),
                        perm=torch.full((T * Kp,), -7, **i32), offsets=torch.full((N + 1,), -7, **i32))
        if gemm_path:
            ex.exfold_moe_prefill_ex(self.layer, self.d_x, self.d_lg, self.d_wg, self.d_wu, self.d_wd, self.tables, Kp, y,
                                     ws, gemm_path=gemm_path, meta=meta)
        else:
            ex.exfold_moe_prefill(self.layer, self.d_x, self.d_lg, self.d_wg, self.d_wu, self.d_wd, self.tables, Kp, y,
                                  ws, meta=meta)
        assert ex.exfold_device_status(ws) == 0
        out = {k: v.cpu().numpy() for k, v in (meta or {}).items()}
        out["y"] = y.float().cpu().numpy()
        return out

    def run_decode(self, M, with_meta=True):
        ex, cfg, B = self.ex, self.cfg, self.B
        K, N = cfg.top_k, cfg.n_experts
        ws = self.workspace(B, K)
        y = torch.full((B, cfg.hidden), float("nan"), dtype=self.d_wg.dtype, device=self.dev)
        meta = None
        if with_meta:
            i32 = dict(dtype=torch.int32, device=self.dev)
            f32 = dict(dtype=torch.float32, device=self.dev)
            meta = dict(pool_ids=torch.full((M,), -7, **i32), pool_size=torch.full((1,), -7, **i32),
                        pool_mask=torch.zeros(((N + 31) // 32,), **i32), ids=torch.full((B, K), -7, **i32),
                        w=torch.full((B, K), float("nan"), **f32), target=torch.full((N,), -7, **i32),
                        scale=torch.full((N,), float("nan"), **f32))
        ex.exfold_moe_decode(self.layer, self.d_xd, self.d_lgd, self.d_wg, self.d_wu, self.d_wd, self.tables, M, y, ws,
                             meta=meta)
        assert ex.exfold_device_status(ws) == 0
        out = {k: v.cpu().numpy() for k, v in (meta or {}).items()}
        out["y"] = y.float().cpu().numpy()
        return out

    # ---------------------------------------------------------------- oracle runs
    def oracle_prefill(self, Kp, tok_idx=None):
        cfg = self.cfg
        S, L, h, lnh = self.np_tables()
        ref = oracle.prefill_fold(self.lg.numpy(), cfg.top_k, Kp, S, L, h, lnh)
        ref["perm"], off = oracle.sort_routes(ref["ids"], cfg.n_experts)
        ref["offsets"] = off
        ref["y"] = oracle.moe_apply(A(self.x), A(self.wg), A(self.wu), A(self.wd), ref["ids"], ref["w"],
                                    cfg.n_experts, cfg.n_shared, tok_idx=tok_idx)
        return ref

    def oracle_decode(self, M):
        cfg = self.cfg
        S, L, h, lnh = self.np_tables()
        ref = oracle.decode_fold(self.lgd.numpy(), cfg.top_k, M, S, L, h)
        ref["y"] = oracle.moe_apply(A(self.xd), A(self.wg), A(self.wu), A(self.wd), ref["ids"], ref["w"],
                                    cfg.n_experts, cfg.n_shared)
        return ref


def check_output(y, yref, dtype):
    """Tolerances of the parity contract: bf16 layers max|err| <= 2e-2 max|ref| and relative Frobenius
    error <= 1e-2; fp32 layers 1e-4 on both."""
    assert np.isfinite(y).all(), "non-finite values (an output row was never written?)"
    tol_max, tol_fro = (2e-2, 1e-2) if dtype == "bf16" else (1e-4, 1e-4)
    scale = np.abs(yref).max()
    err_max = np.abs(y - yref).max() / scale
    err_fro = np.linalg.norm(y - yref) / np.linalg.norm(yref)
    assert err_max <= tol_max, f"max error {err_max:.3e} > {tol_max}"
    assert err_fro <= tol_fro, f"relative Frobenius error {err_fro:.3e} > {tol_fro}"
    return err_max, err_fro


def check_prefill_meta(got, ref):
    """Routing metadata is integer work: bit-exact. Folded weights: fp32 vs double arithmetic."""
    for k in ("ids", "omit_src", "omit_tgt", "perm", "offsets"):
        assert np.array_equal(got[k], ref[k]), f"prefill {k} differs from the oracle"
    np.testing.assert_allclose(got["w"], ref["w"], rtol=1e-5, atol=1e-7)


def check_decode_meta(got, ref, M):
    assert int(got["pool_size"][0]) == ref["pool_size"]
    assert np.array_equal(got["pool_ids"], ref["pool_ids"][:M])
    assert np.array_equal(got["pool_mask"].view(np.uint32), ref["pool_mask"])
    assert np.array_equal(got["ids"], ref["ids"])
    assert np.array_equal(got["target"], ref["target"])
    assert np.array_equal(got["scale"], ref["scale"])
    np.testing.assert_allclose(got["w"], ref["w"], rtol=1e-6, atol=1e-7)
