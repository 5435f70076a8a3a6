"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs. Routing metadata bit-exact, outputs within the stated tolerances."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from harness import A, Case, check_decode_meta, check_output, check_prefill_meta

pytestmark = pytest.mark.gpu

TINY = si.CONFIGS["tiny"]


def small_bf16(**kw):
    base = dict(name="small", n_experts=16, n_shared=0, hidden=256, inter=384, top_k=4, dtype="bf16",
                prefill_tokens=300, k_pre=(2,), decode_batch=24, pool_m=(6,), logits="zipf")
    base.update(kw)
    return si.LayerConfig(**base)


def calibrated_tables(case, cfg, lam=1e-3):
    xc = si.hidden_states(cfg, cfg.calib_tokens, "x_cal")
    lc = si.router_logits(cfg, cfg.calib_tokens, "logits_cal")
    cal = oracle.calibrate(A(xc), lc.numpy(), A(case.wg), A(case.wu), A(case.wd), cfg.n_experts, cfg.top_k, lam=lam)
    return xc, lc, cal


# ------------------------------------------------------------------ fp32 tiny layer (SIMT path)
@pytest.mark.parametrize("correlated", [0.0, 0.8])
def test_tiny_fp32_layer(correlated):
    cfg = TINY
    case = Case(cfg, std=0.02, correlated=correlated)
    xc, lc, cal = calibrated_tables(case, cfg)
    case.set_tables((cal["S"], cal["L"], cal["h"], cal["lnh"]))
    if correlated:
        off = ~np.eye(cfg.n_experts, dtype=bool)
        assert np.abs(cal["S"][off]).mean() > 0.2   # folding matters in this variant
    for Kp in (1, 2):
        got, ref = case.run_prefill(Kp), case.oracle_prefill(Kp)
        check_prefill_meta(got, ref)
        check_output(got["y"], ref["y"], "f32")
    for M in (4, 1, 8):
        got, ref = case.run_decode(M), case.oracle_decode(M)
        assert ref["min_gap"] > 1e-9, "degenerate input: pool boundary tie"
        check_decode_meta(got, ref, M)
        check_output(got["y"], ref["y"], "f32")


@pytest.mark.parametrize("mode", [0, 1])
def test_calibrate_matches_oracle(mode):
    cfg = TINY
    case = Case(cfg, std=0.02, correlated=0.8)
    ex, dev = case.ex, case.dev
    m, N, K = cfg.calib_tokens, cfg.n_experts, cfg.top_k
    xc = si.hidden_states(cfg, m, "x_cal")
    lc = si.router_logits(cfg, m, "logits_cal")
    ref = oracle.calibrate(A(xc), lc.numpy(), A(case.wg), A(case.wu), A(case.wd), N, K, mode=mode)
    S = torch.full((N, N), float("nan"), device=dev)
    L, h, lnh = torch.full_like(S, float("nan")), torch.full((N,), float("nan"), device=dev), torch.empty(N, device=dev)
    n_obs = torch.full((N, N), -1, dtype=torch.int32, device=dev)
    ws = ex.alloc_workspace(case.layer, m, N if mode else K)
    ws.fill_(0xFF)
    rc = ex.exfold_calibrate(case.layer, xc.to(dev), lc.to(dev), case.d_wg, case.d_wu, case.d_wd,
                             ex.make_tables(S, L, h, lnh, n_obs), ws, mode=mode)
    assert rc == (1 if ref["unobserved"] else 0)
    assert np.array_equal(n_obs.cpu().numpy(), ref["n_obs"])
    np.testing.assert_allclose(S.cpu().numpy(), ref["S"], rtol=2e-5, atol=2e-6)
    np.testing.assert_allclose(L.cpu().numpy(), ref["L"], rtol=1e-4, atol=2e-5)
    np.testing.assert_allclose(h.cpu().numpy(), ref["h"], rtol=1e-5)
    np.testing.assert_allclose(lnh.cpu().numpy(), ref["lnh"], rtol=1e-5, atol=1e-6)
    assert (np.diag(S.cpu().numpy()) == 1).all() and (np.diag(L.cpu().numpy()) == 0).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_calibrate_layers_equals_one_call_per_layer(dtype):
    """Three layers (own weights, calibration sets of different lengths) in one call: tables bit-identical to
    those of three exfold_calibrate calls, per-job unobserved counts as returned by the single calls."""
    cfg = TINY if dtype == "f32" else small_bf16(n_experts=8, top_k=2, hidden=128, inter=192, calib_tokens=300)
    cases = [Case(si.scaled(cfg, seed=cfg.seed + j), std=0.02, correlated=0.5) for j in range(3)]
    ex, dev = cases[0].ex, cases[0].dev
    N, K = cfg.n_experts, cfg.top_k
    ms = [cfg.calib_tokens, cfg.calib_tokens // 2 + 3, 40]

    def fresh():
        S = torch.full((N, N), float("nan"), device=dev)
        return dict(S=S, L=torch.full_like(S, float("nan")), h=torch.full((N,), float("nan"), device=dev),
                    lnh=torch.empty(N, device=dev), n_obs=torch.full((N, N), -1, dtype=torch.int32, device=dev))

    inputs = [(si.hidden_states(c.cfg, m, "x_cal").to(dev), si.router_logits(c.cfg, m, "logits_cal").to(dev))
              for c, m in zip(cases, ms)]
    ws = ex.alloc_workspace(cases[0].layer, max(ms), K)
    single, rcs = [], []
    for c, (xc, lc) in zip(cases, inputs):
        t = fresh()
        rcs.append(ex.exfold_calibrate(c.layer, xc, lc, c.d_wg, c.d_wu, c.d_wd,
                                       ex.make_tables(t["S"], t["L"], t["h"], t["lnh"], t["n_obs"]), ws))
        single.append({k: v.cpu().numpy() for k, v in t.items()})
    batched = [fresh() for _ in cases]
    tabs = [ex.make_tables(t["S"], t["L"], t["h"], t["lnh"], t["n_obs"]) for t in batched]
    ws.fill_(0xFF)
    rc, unobserved = ex.exfold_calibrate_layers(
        cases[0].layer, [(xc, lc, c.d_wg, c.d_wu, c.d_wd, tab) for c, (xc, lc), tab in zip(cases, inputs, tabs)], ws)
    assert rc == max(rcs)
    assert [int(u > 0) for u in unobserved] == rcs
    for a, b in zip(single, batched):
        for k in a:
            assert np.array_equal(a[k], b[k].cpu().numpy(), equal_nan=True), k


def test_calibrate_common_input_many_experts_fp32():
    """Common-input mode with N >= 32 takes the Gram-product form of the pair sums; fp32 layer, tight bound."""
    cfg = si.LayerConfig("f32_many", 40, 0, 96, 64, 2, "f32", 64, (1,), 16, (4,))
    case = Case(cfg, std=0.05, correlated=0.8)
    ex, dev = case.ex, case.dev
    m, N, K = 203, cfg.n_experts, cfg.top_k
    xc = si.hidden_states(cfg, m, "x_cal")
    lc = si.router_logits(cfg, m, "logits_cal")
    ref = oracle.calibrate(A(xc), lc.numpy(), A(case.wg), A(case.wu), A(case.wd), N, K, mode=1)
    S = torch.full((N, N), float("nan"), device=dev)
    L, h, lnh = torch.full_like(S, float("nan")), torch.full((N,), float("nan"), device=dev), torch.empty(N, device=dev)
    n_obs = torch.full((N, N), -1, dtype=torch.int32, device=dev)
    ws = ex.alloc_workspace(case.layer, m, N)
    ws.fill_(0xFF)
    rc = ex.exfold_calibrate(case.layer, xc.to(dev), lc.to(dev), case.d_wg, case.d_wu, case.d_wd,
                             ex.make_tables(S, L, h, lnh, n_obs), ws, mode=1)
    assert rc == 0
    assert np.array_equal(n_obs.cpu().numpy(), ref["n_obs"])
    np.testing.assert_allclose(S.cpu().numpy(), ref["S"], rtol=2e-5, atol=2e-6)
    np.testing.assert_allclose(L.cpu().numpy(), ref["L"], rtol=1e-4, atol=2e-5)
    np.testing.assert_allclose(h.cpu().numpy(), ref["h"], rtol=1e-5)


@pytest.mark.parametrize("mode,N", [(0, 16), (1, 16), (1, 40)])
def test_calibrate_bf16_on_tensor_cores(mode, N):
    """bf16 layers calibrate through the grouped tcgen05 GEMMs (Eq. 6-9 on fp32 outputs, H rounded to bf16).

    Tolerance: rounding H to bf16 perturbs every expert output by ~2^-9/sqrt(3) of its norm in a random
    direction, so per-token inner products move by ~1e-3 relative; the tables average many tokens.
    700 tokens = several 128-row tiles per expert plus a ragged tail.
    """
    cfg = small_bf16(n_experts=N)
    case = Case(cfg, correlated=0.8)
    ex, dev = case.ex, case.dev
    m, K = 700, cfg.top_k
    xc = si.hidden_states(cfg, m, "x_cal")
    lc = si.router_logits(cfg, m, "logits_cal")
    ref = oracle.calibrate(A(xc), lc.numpy(), A(case.wg), A(case.wu), A(case.wd), N, K, mode=mode)
    S = torch.full((N, N), float("nan"), device=dev)
    L, h, lnh = torch.full_like(S, float("nan")), torch.full((N,), float("nan"), device=dev), torch.empty(N, device=dev)
    n_obs = torch.full((N, N), -1, dtype=torch.int32, device=dev)
    ws = ex.alloc_workspace(case.layer, m, N if mode else K)
    ws.fill_(0xFF)
    rc = ex.exfold_calibrate(case.layer, xc.to(dev), lc.to(dev), case.d_wg, case.d_wu, case.d_wd,
                             ex.make_tables(S, L, h, lnh, n_obs), ws, mode=mode)
    assert rc == (1 if ref["unobserved"] else 0)
    assert ex.exfold_device_status(ws) == 0
    assert np.array_equal(n_obs.cpu().numpy(), ref["n_obs"])
    Sg, Lg = S.cpu().numpy(), L.cpu().numpy()
    seen = ref["n_obs"] > 0
    off = ~np.eye(N, dtype=bool)
    assert np.abs(ref["S"][off & seen]).mean() > 0.1          # a table worth comparing
    np.testing.assert_allclose(Sg, ref["S"], rtol=5e-3, atol=5e-3)
    np.testing.assert_allclose(Lg[seen | ~off], ref["L"][seen | ~off], rtol=5e-3, atol=5e-3)
    assert (Lg[~seen & off] == np.float32(1e30)).all() and (Sg[~seen & off] == 0).all()
    np.testing.assert_allclose(h.cpu().numpy(), ref["h"], rtol=3e-3)
    np.testing.assert_allclose(lnh.cpu().numpy(), ref["lnh"], rtol=0, atol=3e-3)
    assert (np.diag(Sg) == 1).all() and (np.diag(Lg) == 0).all()


# ------------------------------------------------------------------ bf16 tensor-core path
@pytest.mark.parametrize("Kp", [2, 1, 4])
def test_bf16_prefill_small(Kp):
    case = Case(small_bf16())
    got, ref = case.run_prefill(Kp), case.oracle_prefill(Kp)
    assert ref["mismatch"] == 0
    check_prefill_meta(got, ref)
    check_output(got["y"], ref["y"], "bf16")


@pytest.mark.parametrize("M", [6, 1, 16])
def test_bf16_decode_small(M):
    case = Case(small_bf16())
    got, ref = case.run_decode(M), case.oracle_decode(M)
    assert ref["min_gap"] > 1e-9
    check_decode_meta(got, ref, M)
    check_output(got["y"], ref["y"], "bf16")


def test_bf16_shared_expert_and_correlated_experts():
    cfg = small_bf16(n_shared=1, n_experts=8, top_k=3, prefill_tokens=200, decode_batch=17)
    case = Case(cfg, correlated=0.8)
    got, ref = case.run_prefill(2), case.oracle_prefill(2)
    check_prefill_meta(got, ref)
    check_output(got["y"], ref["y"], "bf16")
    got, ref = case.run_decode(3), case.oracle_decode(3)
    check_decode_meta(got, ref, 3)
    check_output(got["y"], ref["y"], "bf16")


def test_bf16_several_tiles_and_ragged_tail():
    """Groups of 0, 1, hundreds of rows; several 128-row tiles per expert; K and N tails."""
    cfg = small_bf16(n_experts=8, hidden=512, inter=832, top_k=2, prefill_tokens=1111, decode_batch=64,
                     logits="zipf", zipf_s=2.0)
    case = Case(cfg)
    lgm = case.lg.clone()
    lgm[:, 5] = -50.0          # expert 5 receives no route at all
    case.lg, case.d_lg = lgm, lgm.to(case.dev)
    for Kp in (1, 2):
        got, ref = case.run_prefill(Kp), case.oracle_prefill(Kp)
        counts = np.diff(ref["offsets"])
        assert counts[5] == 0 and counts.max() > 256
        check_prefill_meta(got, ref)
        check_output(got["y"], ref["y"], "bf16")
    got, ref = case.run_decode(3), case.oracle_decode(3)
    check_decode_meta(got, ref, 3)
    check_output(got["y"], ref["y"], "bf16")


@pytest.mark.parametrize("shape", ["skewed", "shared", "top1"])
def test_prefill_on_cta_pairs_matches_oracle_and_the_one_cta_kernel(shape):
    """gemm_path = 2 runs every pair of row tiles of a group on the CTA-pair kernel and the odd last tiles on the
    one-CTA kernel, whatever the size; = 1 keeps everything on the one-CTA kernel. Both must match the oracle, and
    each other to the last bit (the same products are accumulated in the same order)."""
    if shape == "skewed":    # groups of 0, 1, 2, 3, ... row tiles, ragged last tiles, K and N tails
        cfg = small_bf16(n_experts=8, hidden=512, inter=832, top_k=2, prefill_tokens=1500, logits="zipf", zipf_s=1.5)
        Kps = (1, 2)
    elif shape == "shared":  # the shared expert's group reads x in place: 7 tiles = 3 pairs + an odd tile
        cfg = small_bf16(n_experts=6, n_shared=1, hidden=320, inter=448, top_k=3, prefill_tokens=777, logits="normal")
        Kps = (2,)
    else:                    # K' = 1 without a shared expert: GEMM-2 writes y directly
        cfg = small_bf16(n_experts=4, hidden=256, inter=256, top_k=2, prefill_tokens=1024, logits="normal")
        Kps = (1,)
    case = Case(cfg)
    for Kp in Kps:
        ref = case.oracle_prefill(Kp)
        got_pair = case.run_prefill(Kp, gemm_path=2)
        got_one = case.run_prefill(Kp, gemm_path=1)
        counts = np.diff(ref["offsets"])
        assert counts.max() >= 256          # at least one whole pair of row tiles
        check_prefill_meta(got_pair, ref)
        check_output(got_pair["y"], ref["y"], "bf16")
        check_output(got_one["y"], ref["y"], "bf16")
        assert np.array_equal(got_pair["y"], got_one["y"])   # bf16 values widened to float32: exact comparison


def test_prefill_with_side_by_side_passes_replays_from_a_cuda_graph():
    """A prefill call whose GEMMs fork onto the library's second stream is captured into a CUDA graph (the fork and
    the join are events on the capturing stream) and replays to the same bits as the direct call."""
    cfg = small_bf16(n_experts=4, hidden=256, inter=256, top_k=2, prefill_tokens=2048, logits="normal")  # 32 row tiles
    case = Case(cfg)
    ex, T = case.ex, cfg.prefill_tokens
    ws = case.workspace(T, 2)
    y_direct = torch.empty((T, cfg.hidden), dtype=case.d_wg.dtype, device=case.dev)
    y_graph = torch.full_like(y_direct, float("nan"))
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for y in (y_direct, y_direct):   # the second call runs with every lazily created object in place
            ex.exfold_moe_prefill(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, 2, y, ws,
                                  stream=stream)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ex.exfold_moe_prefill(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, 2, y_graph,
                                  ws, stream=stream)
        for _ in range(3):
            graph.replay()
        stream.synchronize()
    assert ex.exfold_device_status(ws) == 0
    assert torch.equal(y_direct.view(torch.int16), y_graph.view(torch.int16))
    ref = case.oracle_prefill(2)
    check_output(y_graph.float().cpu().numpy(), ref["y"], "bf16")


@pytest.mark.parametrize("T", [1, 63, 129])
def test_bf16_odd_token_counts(T):
    cfg = small_bf16(prefill_tokens=T, decode_batch=min(T, 256))
    case = Case(cfg)
    got, ref = case.run_prefill(2), case.oracle_prefill(2)
    check_prefill_meta(got, ref)
    check_output(got["y"], ref["y"], "bf16")
    got, ref = case.run_decode(4), case.oracle_decode(4)
    check_decode_meta(got, ref, 4)
    check_output(got["y"], ref["y"], "bf16")


def test_full_budget_is_the_unfolded_layer():
    """K' = K and M = N: no folding, output equals Eq. 3 computed by the oracle from Eq. 2's routes."""
    cfg = small_bf16()
    case = Case(cfg)
    ids, w, _ = oracle.gate(case.lg.numpy(), cfg.top_k)
    y_unf = oracle.moe_apply(A(case.x), A(case.wg), A(case.wu), A(case.wd), ids, w, cfg.n_experts)
    got = case.run_prefill(cfg.top_k)
    assert np.array_equal(np.sort(got["ids"], 1), np.sort(ids, 1))
    check_output(got["y"], y_unf, "bf16")
    idd, wd_, _ = oracle.gate(case.lgd.numpy(), cfg.top_k)
    yd_unf = oracle.moe_apply(A(case.xd), A(case.wg), A(case.wu), A(case.wd), idd, wd_, cfg.n_experts)
    gotd = case.run_decode(cfg.n_experts)
    assert np.array_equal(gotd["ids"], idd)
    np.testing.assert_allclose(gotd["w"], wd_, rtol=1e-6)
    check_output(gotd["y"], yd_unf, "bf16")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_maximum_expert_count_and_top_k(dtype):
    """N = 256 experts and K = 32 routes per token are the limits of the interface."""
    cfg = small_bf16(n_experts=256, top_k=32, hidden=128, inter=128, dtype=dtype, prefill_tokens=150,
                     decode_batch=40, logits="normal")
    case = Case(cfg)
    for Kp in (8, 31):
        got, ref = case.run_prefill(Kp), case.oracle_prefill(Kp)
        assert ref["mismatch"] == 0
        check_prefill_meta(got, ref)
        check_output(got["y"], ref["y"], dtype)
    for M in (64, 256):
        got, ref = case.run_decode(M), case.oracle_decode(M)
        assert ref["min_gap"] > 1e-9
        check_decode_meta(got, ref, M)
        check_output(got["y"], ref["y"], dtype)


def test_decode_max_batch_and_all_unobserved_row():
    cfg = small_bf16(n_experts=32, top_k=8, decode_batch=256, prefill_tokens=64)
    case = Case(cfg)
    S, L, h, lnh = [t.clone() for t in case.tables_host]
    L[3, :] = 1e30
    L[3, 3] = 0.0
    S[3, :] = 0.0
    S[3, 3] = 1.0
    case.set_tables((S, L, h, lnh))
    for M in (8, 20):
        got, ref = case.run_decode(M), case.oracle_decode(M)
        assert ref["min_gap"] > 1e-9
        check_decode_meta(got, ref, M)
        check_output(got["y"], ref["y"], "bf16")
    got, ref = case.run_prefill(3), case.oracle_prefill(3)
    check_prefill_meta(got, ref)
    check_output(got["y"], ref["y"], "bf16")


@pytest.mark.parametrize("n_shared,M", [(0, 5), (1, 3), (0, 16)])
def test_static_pool_decode(n_shared, M):
    """Static pool built on the GPU equals the oracle's; a decode step with it equals the per-route
    remap followed by the expert FFN."""
    cfg = small_bf16(n_shared=n_shared, decode_batch=40)
    case = Case(cfg)
    ex, dev = case.ex, case.dev
    N, K, B = cfg.n_experts, cfg.top_k, case.B
    S, L, h, lnh = case.np_tables()
    ref_pool = oracle.static_pool(M, S, L, h)
    pool_ids = torch.full((M,), -7, dtype=torch.int32, device=dev)
    target = torch.full((N,), -7, dtype=torch.int32, device=dev)
    scale = torch.full((N,), float("nan"), dtype=torch.float32, device=dev)
    sp = ex.exfold_static_pool_build(case.layer, case.tables, M, pool_ids, target, scale)
    torch.cuda.synchronize()
    assert np.array_equal(pool_ids.cpu().numpy(), ref_pool["pool_ids"])
    assert np.array_equal(target.cpu().numpy(), ref_pool["target"])
    assert np.array_equal(scale.cpu().numpy(), ref_pool["scale"])
    ref = oracle.decode_static(case.lgd.numpy(), K, ref_pool["target"], ref_pool["scale"])
    yref = oracle.moe_apply(A(case.xd), A(case.wg), A(case.wu), A(case.wd), ref["ids"], ref["w"], N, n_shared)
    ws = case.workspace(B, K)
    y = torch.full((B, cfg.hidden), float("nan"), dtype=torch.bfloat16, device=dev)
    meta = dict(ids=torch.full((B, K), -7, dtype=torch.int32, device=dev),
                w=torch.full((B, K), float("nan"), dtype=torch.float32, device=dev),
                pool_ids=torch.full((M,), -7, dtype=torch.int32, device=dev))
    for _ in range(2):
        ex.exfold_moe_decode_static(case.layer, case.d_xd, case.d_lgd, case.d_wg, case.d_wu, case.d_wd, sp, y, ws,
                                    meta=meta)
        assert ex.exfold_device_status(ws) == 0
        assert np.array_equal(meta["ids"].cpu().numpy(), ref["ids"])
        np.testing.assert_allclose(meta["w"].cpu().numpy(), ref["w"], rtol=1e-6, atol=1e-7)
        assert np.array_equal(meta["pool_ids"].cpu().numpy(), ref_pool["pool_ids"])
        check_output(y.float().cpu().numpy(), yref, "bf16")


@pytest.mark.parametrize("thr,rescale,conf", [(0.6, False, False), (0.6, True, False), (float("inf"), False, True),
                                              (0.5, True, True), (-1.0, True, False)])
def test_prefill_safeguards(thr, rescale, conf):
    cfg = small_bf16(n_experts=32, top_k=6, prefill_tokens=500, hidden=128, inter=128)
    case = Case(cfg)
    ex, dev, T, K, Kp = case.ex, case.dev, case.T, cfg.top_k, 3
    S, L, h, lnh = case.np_tables()
    ref = oracle.prefill_fold_safe(case.lg.numpy(), K, Kp, S, L, lnh, loss_thr=thr, rescale=rescale, confidence=conf)
    yref = oracle.moe_apply(A(case.x), A(case.wg), A(case.wu), A(case.wd), ref["ids"], ref["w"], cfg.n_experts)
    ws = case.workspace(T, Kp)
    y = torch.full((T, cfg.hidden), float("nan"), dtype=torch.bfloat16, device=dev)
    i32 = dict(dtype=torch.int32, device=dev)
    meta = dict(ids=torch.full((T, Kp), -7, **i32), w=torch.full((T, Kp), float("nan"), device=dev),
                omit_src=torch.full((T, K - Kp), -7, **i32), omit_tgt=torch.full((T, K - Kp), -7, **i32))
    ex.exfold_moe_prefill_ex(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, Kp, y, ws,
                             loss_threshold=thr, rescale=rescale, confidence_split=conf, meta=meta)
    assert ex.exfold_device_status(ws) == 0
    for k in ("ids", "omit_src", "omit_tgt"):
        assert np.array_equal(meta[k].cpu().numpy(), ref[k]), k
    np.testing.assert_allclose(meta["w"].cpu().numpy(), ref["w"], rtol=2e-5, atol=2e-5)
    check_output(y.float().cpu().numpy(), yref, "bf16")


def test_results_are_reproducible_and_meta_is_optional():
    case = Case(small_bf16())
    a = case.run_prefill(2)
    b = case.run_prefill(2)
    for k in ("ids", "perm", "offsets", "omit_src", "omit_tgt"):
        assert np.array_equal(a[k], b[k])
    assert np.array_equal(a["w"], b["w"])
    c = case.run_prefill(2, with_meta=False)
    np.testing.assert_allclose(c["y"], a["y"], rtol=0, atol=2e-2 * np.abs(a["y"]).max())
    d1, d2 = case.run_decode(6), case.run_decode(6, with_meta=False)
    assert np.array_equal(d2["y"], d1["y"])   # no atomics on the decode path either: bit for bit


def test_device_status_record_is_decoded_and_cleared():
    """The status record at the start of the workspace: a code written there (here from the host, never
    by faulting a kernel) is reported once by exfold_device_status and cleared; every call clears it first."""
    case = Case(small_bf16())
    ex = case.ex
    ws = case.workspace(case.T, 2)
    ws[:256].zero_()
    assert ex.exfold_device_status(ws) == ex.EXFOLD_OK
    ws[:4].copy_(torch.tensor([ex.EXFOLD_ERR_DEVICE_TIMEOUT], dtype=torch.int32).view(torch.uint8))
    assert ex.exfold_device_status(ws) == ex.EXFOLD_ERR_DEVICE_TIMEOUT
    assert ex.exfold_device_status(ws) == ex.EXFOLD_OK
    ws[:4].copy_(torch.tensor([-77], dtype=torch.int32).view(torch.uint8))      # unknown code
    assert ex.exfold_device_status(ws) == ex.EXFOLD_ERR_CUDA
    ws[:4].copy_(torch.tensor([ex.EXFOLD_ERR_DEVICE_TIMEOUT], dtype=torch.int32).view(torch.uint8))
    y = torch.empty((case.T, case.cfg.hidden), dtype=torch.bfloat16, device=case.dev)
    ex.exfold_moe_prefill(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, 2, y, ws)
    assert ex.exfold_device_status(ws) == ex.EXFOLD_OK    # a stale code does not survive the next call


def test_host_buffer_entry_points():
    case = Case(small_bf16())
    ex, cfg = case.ex, case.cfg
    T, B, K = case.T, case.B, cfg.top_k
    ws = ex.alloc_workspace(case.layer, max(T, B), K, host_staging=True)
    xh, lh = case.x.pin_memory(), case.lg.pin_memory()
    yh = torch.empty((T, cfg.hidden), dtype=torch.bfloat16).pin_memory()
    ex.exfold_moe_prefill_host(case.layer, xh, lh, case.d_wg, case.d_wu, case.d_wd, case.tables, 2, yh, ws)
    assert ex.exfold_device_status(ws) == 0
    ref = case.oracle_prefill(2)
    check_output(yh.float().numpy(), ref["y"], "bf16")
    xdh, ldh = case.xd.pin_memory(), case.lgd.pin_memory()
    ydh = torch.empty((B, cfg.hidden), dtype=torch.bfloat16).pin_memory()
    ex.exfold_moe_decode_host(case.layer, xdh, ldh, case.d_wg, case.d_wu, case.d_wd, case.tables, 6, ydh, ws)
    assert ex.exfold_device_status(ws) == 0
    check_output(ydh.float().numpy(), case.oracle_decode(6)["y"], "bf16")


# ------------------------------------------------------------------ router scores (input of Eq. 2)
@pytest.mark.parametrize("dtype,N,T", [("bf16", 16, 300), ("bf16", 8, 129), ("bf16", 200, 1000), ("bf16", 6, 277),
                                       ("bf16", 6, 77), ("bf16", 128, 64), ("f32", 8, 64)])
def test_router_logits_match_oracle(dtype, N, T):
    """logits = x W_r^T on the tensor cores (bf16) / fp32 dot products: within 1e-4 of the largest score.
    N = 8 and 6 end inside the first 32-column chunk (6: rows not 16-byte aligned), N = 200 spans seven; batches of
    at most 128 tokens take the dot-product kernel also for bf16."""
    cfg = small_bf16(n_experts=N, top_k=2, dtype=dtype, prefill_tokens=T, hidden=256 if dtype == "bf16" else 128)
    ex = Case(cfg).ex
    dev = torch.device("cuda:0")
    x, wr = si.hidden_states(cfg, T), si.router_weights(cfg)
    ref32, _ = oracle.router_logits(A(x), A(wr))
    layer = ex.make_layer(N, 0, cfg.hidden, cfg.inter, cfg.top_k, cfg.dtype)
    ws = ex.alloc_workspace(layer, T, 1)
    ws.fill_(0xFF)
    lg = torch.full((T, N), float("nan"), device=dev)
    assert ex.exfold_router_logits(layer, x.to(dev), wr.to(dev), lg, ws) == 0
    assert ex.exfold_device_status(ws) == 0
    got = lg.cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - ref32).max() <= 1e-4 * np.abs(ref32).max()


def test_router_then_prefill_chain():
    """Scores from the GPU router feed the folded prefill; the oracle runs its own scores through its own layer.
    Tokens whose ranking-relevant gaps (between the Top-(K+1) scores, and between retained-set keys) exceed the
    accumulation error must agree bit for bit in routing; the outputs of those tokens agree to the bf16 bound."""
    cfg = small_bf16(n_experts=16, top_k=4, prefill_tokens=400)
    case = Case(cfg)
    ex, dev = case.ex, case.dev
    T, N, K, Kp = 400, 16, 4, 2
    wr = si.router_weights(cfg)
    ref32, ref64 = oracle.router_logits(A(case.x), A(wr))
    ws = ex.alloc_workspace(case.layer, T, K)
    lg = torch.empty((T, N), device=dev)
    assert ex.exfold_router_logits(case.layer, case.d_x, wr.to(dev), lg, ws) == 0
    got_lg = lg.cpu().numpy()
    tol = 1e-4 * np.abs(ref32).max()
    assert np.abs(got_lg - ref32).max() <= tol
    # tokens that are safe against a perturbation of every score by tol
    lnh = case.tables_host[3].numpy()
    srt = np.sort(ref64, axis=1)[:, ::-1]
    gap_topk = (srt[:, :K] - srt[:, 1:K + 1]).min(axis=1)
    ids_ref, _, _ = oracle.gate(ref32, K)
    keys = np.take_along_axis(ref64, ids_ref.astype(np.int64), 1) + lnh[ids_ref]
    ks = np.sort(keys, axis=1)[:, ::-1]
    gap_keys = (ks[:, :-1] - ks[:, 1:]).min(axis=1)
    safe = (gap_topk > 4 * tol) & (gap_keys > 4 * tol)
    assert safe.mean() > 0.9
    case.lg, case.d_lg = torch.from_numpy(ref32), lg      # oracle side: its own scores; GPU side: the GPU's
    ref = case.oracle_prefill(Kp)
    got = case.run_prefill(Kp)
    assert np.array_equal(got["ids"][safe], ref["ids"][safe])
    assert np.array_equal(got["omit_tgt"][safe], ref["omit_tgt"][safe])
    np.testing.assert_allclose(got["w"][safe], ref["w"][safe], rtol=2e-3, atol=1e-5)
    check_output(got["y"][safe], ref["y"][safe], "bf16")


def test_host_prefill_in_chunks_equals_the_device_call():
    """4096+ tokens without metadata go through the host-buffer call in overlapped chunks (ragged last chunk):
    same bits as one device call; with metadata the call is not split and the routing still matches the oracle."""
    cfg = small_bf16(n_experts=8, hidden=128, inter=128, top_k=2, prefill_tokens=4500, decode_batch=8)
    case = Case(cfg)
    ex, T = case.ex, case.T
    ref_dev = case.run_prefill(1, with_meta=False)["y"]
    ws = ex.alloc_workspace(case.layer, T, cfg.top_k, host_staging=True)
    xh, lh = case.x.pin_memory(), case.lg.pin_memory()
    yh = torch.full((T, cfg.hidden), float("nan"), dtype=torch.bfloat16).pin_memory()
    for _ in range(2):  # twice in a row on the same staging buffers
        yh.fill_(float("nan"))
        assert ex.exfold_moe_prefill_host(case.layer, xh, lh, case.d_wg, case.d_wu, case.d_wd, case.tables, 1, yh, ws) == 0
        assert ex.exfold_device_status(ws) == 0
        assert np.array_equal(yh.float().numpy(), ref_dev)
    check_output(ref_dev[:256], case.oracle_prefill(1, tok_idx=np.arange(256))["y"], "bf16")


# ------------------------------------------------------------------ seeded random shapes
def _random_cfg(i):
    """Shape i of a fixed, seeded family: odd expert counts, ragged token counts, every K' and M regime."""
    rng = np.random.default_rng(1000 + i)
    dtype = "bf16" if i % 4 != 3 else "f32"
    N = int(rng.choice([3, 5, 8, 12, 24, 40, 64, 100]))
    K = int(rng.integers(1, min(N, 9) + 1))
    hidden = int(rng.choice([64, 128, 192, 320])) if dtype == "bf16" else int(rng.choice([32, 60, 100]))
    inter = int(rng.choice([64, 128, 448])) if dtype == "bf16" else int(rng.choice([24, 50]))
    T = int(rng.integers(1, 700))
    B = int(rng.integers(1, 257)) if N * 1 else 1
    while B * K > 4096:
        B //= 2
    return si.LayerConfig(f"rand{i}", N, int(rng.integers(0, 2)), hidden, inter, K, dtype, T, (1,), B, (1,),
                          logits="zipf" if rng.random() < 0.5 else "normal", zipf_s=float(rng.choice([0.8, 1.1, 2.0])),
                          seed=20260824 + i)


@pytest.mark.parametrize("i", range(12))
def test_random_shapes(i):
    cfg = _random_cfg(i)
    rng = np.random.default_rng(2000 + i)
    case = Case(cfg, correlated=0.8 if i % 3 == 0 else 0.0)
    Kp = int(rng.integers(1, cfg.top_k + 1))
    got, ref = case.run_prefill(Kp), case.oracle_prefill(Kp)
    assert ref["mismatch"] == 0  # the fp32 key and the fp64 product rank alike on these seeds
    check_prefill_meta(got, ref)
    check_output(got["y"], ref["y"], cfg.dtype)
    M = int(rng.integers(1, cfg.n_experts + 1))
    got, ref = case.run_decode(M), case.oracle_decode(M)
    assert ref["min_gap"] > 1e-9   # no tie at the pool boundary on these seeds
    check_decode_meta(got, ref, M)
    check_output(got["y"], ref["y"], cfg.dtype)
