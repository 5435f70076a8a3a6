"""GPU parity cases beyond the seeded-random ones: exact ties (the "lower expert id wins" reading), the
safeguards / static pool / router scores at the full Qwen3-30B-A3B shape, host-buffer calls that ask for
metadata, and two prefill calls issued by one host thread on two streams."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from harness import A, Case, check_decode_meta, check_output, check_prefill_meta

pytestmark = pytest.mark.gpu


def small_bf16(**kw):
    base = dict(name="edge", n_experts=16, n_shared=0, hidden=256, inter=384, top_k=4, dtype="bf16",
                prefill_tokens=300, k_pre=(2,), decode_batch=24, pool_m=(6,), logits="zipf")
    base.update(kw)
    return si.LayerConfig(**base)


def sample_tokens(T, n, seed=3):
    return np.sort(np.random.default_rng(seed).choice(T, size=min(n, T), replace=False)).astype(np.int64)


# ------------------------------------------------------------------ exact ties
@pytest.mark.parametrize("N,K,Kp", [(16, 4, 2), (40, 8, 3), (128, 8, 4)])
def test_ties_resolve_to_the_lower_expert_id(N, K, Kp):
    """Router logits quantised to a handful of values put exact ties on the Top-K boundary of most tokens; ln h
    quantised to the same grid makes ranking keys (logit + ln h) of different experts coincide exactly, and a loss
    table with few distinct values ties the arg-min of the target search. Every one of those decisions must come
    out as the oracle's (lower id wins): ids, omitted pairs, permutation and offsets bit for bit. Decode ranks the
    pool on h (continuous here), so its boundary is not tied and the same logits exercise the tied Top-K there."""
    cfg = small_bf16(n_experts=N, top_k=K, prefill_tokens=700, decode_batch=48, logits="normal")
    rng = np.random.default_rng(99 + N)
    S, L, h, lnh = [t.numpy().copy() for t in si.synthetic_tables(cfg)]
    lnh = (np.round(rng.uniform(0.0, 1.0, size=N) * 4) / 4).astype(np.float32)      # 0, .25, .. 1
    L = (np.round(L.clip(0, 1) * 3) / 3).astype(np.float32)                           # four loss levels
    np.fill_diagonal(L, 0.0)
    case = Case(cfg, tables=(S, L, h, lnh))
    q = lambda a: torch.from_numpy((np.round(a.numpy() * 2) / 2).astype(np.float32))  # multiples of 0.5
    case.lg, case.lgd = q(case.lg), q(case.lgd)
    case.d_lg, case.d_lgd = case.lg.to(case.dev), case.lgd.to(case.dev)
    lg = case.lg.numpy()
    srt = np.sort(lg, axis=1)[:, ::-1]
    assert (srt[:, K - 1] == srt[:, K]).mean() > 0.3, "the inputs must tie at the Top-K boundary"
    ref = case.oracle_prefill(Kp)
    keys = np.sort(np.take_along_axis(lg, oracle.gate(lg, K)[0].astype(np.int64), 1) + lnh[oracle.gate(lg, K)[0]], 1)
    assert (np.diff(keys, axis=1) == 0).any(axis=1).mean() > 0.3, "ranking keys must tie inside a token's Top-K"
    got = case.run_prefill(Kp)
    check_prefill_meta(got, ref)
    check_output(got["y"], ref["y"], "bf16")
    M = max(2, N // 4)
    ref = case.oracle_decode(M)
    assert ref["min_gap"] > 1e-9
    got = case.run_decode(M)
    check_decode_meta(got, ref, M)
    check_output(got["y"], ref["y"], "bf16")


# ------------------------------------------------------------------ full Qwen3-30B-A3B shape: the other entry points
@pytest.fixture(scope="module")
def qwen3_case():
    return Case(si.CONFIGS["qwen3"], std=0.02)


def test_safeguards_at_the_qwen3_shape(qwen3_case):
    case = qwen3_case
    cfg, ex, dev = case.cfg, case.ex, case.dev
    T, K, Kp, N = case.T, cfg.top_k, 4, cfg.n_experts
    S, L, h, lnh = case.np_tables()
    idx = sample_tokens(T, 64)
    for thr, rescale, conf in ((0.7, True, False), (float("inf"), False, True)):
        ref = oracle.prefill_fold_safe(case.lg.numpy(), K, Kp, S, L, lnh, loss_thr=thr, rescale=rescale, confidence=conf)
        yref = oracle.moe_apply(A(case.x), A(case.wg), A(case.wu), A(case.wd), ref["ids"], ref["w"], N, tok_idx=idx)
        ws = case.workspace(T, Kp)
        y = torch.full((T, cfg.hidden), float("nan"), dtype=torch.bfloat16, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        meta = dict(ids=torch.full((T, Kp), -7, **i32), w=torch.full((T, Kp), float("nan"), device=dev),
                    omit_src=torch.full((T, K - Kp), -7, **i32), omit_tgt=torch.full((T, K - Kp), -7, **i32))
        ex.exfold_moe_prefill_ex(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, Kp, y,
                                 ws, loss_threshold=thr, rescale=rescale, confidence_split=conf, meta=meta)
        assert ex.exfold_device_status(ws) == 0
        for k in ("ids", "omit_src", "omit_tgt"):
            assert np.array_equal(meta[k].cpu().numpy(), ref[k]), k
        np.testing.assert_allclose(meta["w"].cpu().numpy(), ref["w"], rtol=2e-5, atol=2e-5)
        check_output(y.float().cpu().numpy()[idx], yref, "bf16")


def test_static_pool_decode_at_the_qwen3_shape(qwen3_case):
    case = qwen3_case
    cfg, ex, dev = case.cfg, case.ex, case.dev
    N, K, B, M = cfg.n_experts, cfg.top_k, case.B, 32
    S, L, h, lnh = case.np_tables()
    ref_pool = oracle.static_pool(M, S, L, h)
    i32 = dict(dtype=torch.int32, device=dev)
    pool_ids, target = torch.full((M,), -7, **i32), torch.full((N,), -7, **i32)
    scale = torch.full((N,), float("nan"), dtype=torch.float32, device=dev)
    sp = ex.exfold_static_pool_build(case.layer, case.tables, M, pool_ids, target, scale)
    ref = oracle.decode_static(case.lgd.numpy(), K, ref_pool["target"], ref_pool["scale"])
    yref = oracle.moe_apply(A(case.xd), A(case.wg), A(case.wu), A(case.wd), ref["ids"], ref["w"], N, 0)
    ws = case.workspace(B, K)
    y = torch.full((B, cfg.hidden), float("nan"), dtype=torch.bfloat16, device=dev)
    meta = dict(ids=torch.full((B, K), -7, **i32), w=torch.full((B, K), float("nan"), dtype=torch.float32, device=dev))
    ex.exfold_moe_decode_static(case.layer, case.d_xd, case.d_lgd, case.d_wg, case.d_wu, case.d_wd, sp, y, ws, meta=meta)
    assert ex.exfold_device_status(ws) == 0
    assert np.array_equal(pool_ids.cpu().numpy(), ref_pool["pool_ids"])
    assert np.array_equal(target.cpu().numpy(), ref_pool["target"])
    assert np.array_equal(meta["ids"].cpu().numpy(), ref["ids"])
    np.testing.assert_allclose(meta["w"].cpu().numpy(), ref["w"], rtol=1e-6, atol=1e-7)
    check_output(y.float().cpu().numpy(), yref, "bf16")


def test_router_scores_at_the_qwen3_shape(qwen3_case):
    """8192 tokens x 128 experts on the tensor-core router; the decode batch on the dot-product kernel."""
    case = qwen3_case
    cfg, ex, dev = case.cfg, case.ex, case.dev
    wr = si.router_weights(cfg)
    for x, d_x in ((case.x, case.d_x), (case.xd, case.d_xd)):
        T = x.shape[0]
        ref32, _ = oracle.router_logits(A(x), A(wr))
        ws = case.workspace(T, 1)
        lg = torch.full((T, cfg.n_experts), float("nan"), device=dev)
        assert ex.exfold_router_logits(case.layer, d_x, wr.to(dev), lg, ws) == 0
        assert ex.exfold_device_status(ws) == 0
        got = lg.cpu().numpy()
        assert np.isfinite(got).all()
        assert np.abs(got - ref32).max() <= 1e-4 * np.abs(ref32).max()


# ------------------------------------------------------------------ host-buffer calls that ask for metadata
def test_host_buffer_calls_with_metadata():
    cfg = small_bf16(prefill_tokens=4400, n_experts=8, hidden=128, inter=128, top_k=2)   # long enough to be chunked
    case = Case(cfg)                                                                      # if no metadata is asked
    ex, dev = case.ex, case.dev
    T, B, K, N, Kp, M = case.T, case.B, cfg.top_k, cfg.n_experts, 1, 3
    ws = ex.alloc_workspace(case.layer, max(T, B), K, host_staging=True)
    ws.fill_(0xFF)
    i32 = dict(dtype=torch.int32, device=dev)
    xh, lh = case.x.pin_memory(), case.lg.pin_memory()
    yh = torch.full((T, cfg.hidden), float("nan"), dtype=torch.bfloat16).pin_memory()
    meta = dict(ids=torch.full((T, Kp), -7, **i32), w=torch.full((T, Kp), float("nan"), device=dev),
                omit_src=torch.full((T, K - Kp), -7, **i32), omit_tgt=torch.full((T, K - Kp), -7, **i32),
                perm=torch.full((T * Kp,), -7, **i32), offsets=torch.full((N + 1,), -7, **i32))
    ex.exfold_moe_prefill_host(case.layer, xh, lh, case.d_wg, case.d_wu, case.d_wd, case.tables, Kp, yh, ws, meta=meta)
    assert ex.exfold_device_status(ws) == 0
    ref = case.oracle_prefill(Kp)
    got = {k: v.cpu().numpy() for k, v in meta.items()}
    check_prefill_meta(got, ref)
    check_output(yh.float().numpy(), ref["y"], "bf16")
    xdh, ldh = case.xd.pin_memory(), case.lgd.pin_memory()
    ydh = torch.full((B, cfg.hidden), float("nan"), dtype=torch.bfloat16).pin_memory()
    f32 = dict(dtype=torch.float32, device=dev)
    dmeta = dict(pool_ids=torch.full((M,), -7, **i32), pool_size=torch.full((1,), -7, **i32),
                 pool_mask=torch.zeros(((N + 31) // 32,), **i32), ids=torch.full((B, K), -7, **i32),
                 w=torch.full((B, K), float("nan"), **f32), target=torch.full((N,), -7, **i32),
                 scale=torch.full((N,), float("nan"), **f32))
    ex.exfold_moe_decode_host(case.layer, xdh, ldh, case.d_wg, case.d_wu, case.d_wd, case.tables, M, ydh, ws, meta=dmeta)
    assert ex.exfold_device_status(ws) == 0
    dref = case.oracle_decode(M)
    check_decode_meta({k: v.cpu().numpy() for k, v in dmeta.items()}, dref, M)
    check_output(ydh.float().numpy(), dref["y"], "bf16")


# ------------------------------------------------------------------ one host thread, two streams
def test_two_prefill_calls_on_two_streams_of_one_thread():
    """Calls of >= 24 row tiles run part of their work on a second stream that the library keeps per host
    thread; two caller streams used from one thread share it. Each call has its own workspace and output;
    both must equal the single-stream result bit for bit, and the oracle within tolerance."""
    cfg = small_bf16(n_experts=4, hidden=256, inter=256, top_k=2, prefill_tokens=2048, logits="normal")  # 32 row tiles
    case = Case(cfg)
    ex, T, dev = case.ex, cfg.prefill_tokens, case.dev
    y_ref = case.run_prefill(2, with_meta=False)["y"]
    need = ex.exfold_workspace_bytes(case.layer, T, 2)
    wss = [torch.full((need,), 0xFF, dtype=torch.uint8, device=dev) for _ in range(2)]
    ys = [torch.full((T, cfg.hidden), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for rep in range(3):
        for i in (0, 1):
            ex.exfold_moe_prefill(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, 2,
                                  ys[i], wss[i], stream=streams[i])
    for i in (0, 1):
        assert ex.exfold_device_status(wss[i], streams[i]) == 0
        assert np.array_equal(ys[i].float().cpu().numpy(), y_ref)
    check_output(y_ref, case.oracle_prefill(2)["y"], "bf16")
    assert ex.exfold_thread_release() == 0      # and the per-thread objects come back on the next call
    ex.exfold_moe_prefill(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, 2, ys[0],
                          wss[0])
    assert ex.exfold_device_status(wss[0]) == 0
    assert np.array_equal(ys[0].float().cpu().numpy(), y_ref)


# ------------------------------------------------------------------ layer calls (router matrix in) on an fp32 layer
def test_layer_calls_on_an_fp32_layer():
    """fp32 layers take the separate dot-product router kernel and the SIMT expert path behind the same entry points."""
    cfg = si.CONFIGS["tiny"]
    case = Case(cfg)
    ex, dev = case.ex, case.dev
    T, B, K, N = case.T, case.B, cfg.top_k, cfg.n_experts
    wr = si.router_weights(cfg, std=2.0 / np.sqrt(cfg.hidden))
    S, L, h, lnh = case.np_tables()
    ws = case.workspace(max(T, B), K)
    for x, d_x, n, decode in ((case.x, case.d_x, T, False), (case.xd, case.d_xd, B, True)):
        r32, r64 = oracle.router_logits(A(x), A(wr))
        srt = np.sort(r64, axis=1)[:, ::-1]
        assert (srt[:, :K] - srt[:, 1:K + 1]).min() > 1e-4, "seeded scores without near-ties"
        lg = torch.full((n, N), float("nan"), device=dev)
        y = torch.full((n, cfg.hidden), float("nan"), dtype=torch.float32, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        if decode:
            meta = dict(ids=torch.full((n, K), -7, **i32))
            ex.exfold_moe_decode_layer(case.layer, d_x, wr.to(dev), case.d_wg, case.d_wu, case.d_wd, case.tables, 4, y,
                                       ws, logits_out=lg, meta=meta)
            ref = oracle.decode_fold(r32, K, 4, S, L, h)
        else:
            meta = dict(ids=torch.full((n, 1), -7, **i32))
            ex.exfold_moe_prefill_layer(case.layer, d_x, wr.to(dev), case.d_wg, case.d_wu, case.d_wd, case.tables, 1, y,
                                        ws, logits_out=lg, meta=meta)
            ref = oracle.prefill_fold(r32, K, 1, S, L, h, lnh)
        assert ex.exfold_device_status(ws) == 0
        assert np.abs(lg.cpu().numpy() - r32).max() <= 1e-5 * np.abs(r32).max()
        assert np.array_equal(meta["ids"].cpu().numpy(), ref["ids"])
        yref = oracle.moe_apply(A(x), A(case.wg), A(case.wu), A(case.wd), ref["ids"], ref["w"], N, cfg.n_shared)
        # the weights come from scores that differ in the last bits: looser than the same-logits fp32 bound
        assert np.abs(y.cpu().numpy() - yref).max() <= 1e-3 * np.abs(yref).max()


# ------------------------------------------------------------------ a long prompt: many super-blocks of route blocks
@pytest.mark.parametrize("T,kw", [(150_001, dict(n_experts=8, top_k=2, k_pre=(1,), hidden=64, inter=64)),
                                  (70_000, dict(n_experts=40, n_shared=1, top_k=4, k_pre=(2,), hidden=64, inter=128))])
def test_long_prompt_sorted_routes(T, kw):
    """The sorted position of a route is (rows of lower experts) + (rows of its expert in earlier route blocks);
    the scatter kernel takes both from two levels of histograms (per block of 32 tokens, per super-block of 64 blocks).
    150 001 tokens are 4688 blocks in 74 super-blocks with a ragged last block: permutation, offsets and retained
    experts bit-exact against the oracle's stable sort, outputs on a token sample."""
    case = Case(small_bf16(prefill_tokens=T, decode_batch=8, logits="zipf", **kw), std=0.2)
    cfg, Kp = case.cfg, case.cfg.k_pre[0]
    got = case.run_prefill(Kp)
    S, L, h, lnh = case.np_tables()
    ref = oracle.prefill_fold(case.lg.numpy(), cfg.top_k, Kp, S, L, h, lnh)
    perm, off = oracle.sort_routes(ref["ids"], cfg.n_experts)
    assert np.array_equal(got["ids"], ref["ids"])
    assert np.array_equal(got["offsets"], off)
    assert np.array_equal(got["perm"], perm)
    idx = np.concatenate([sample_tokens(T, 48), np.array([0, T - 1])])
    idx = np.unique(idx)
    yref = oracle.moe_apply(A(case.x), A(case.wg), A(case.wu), A(case.wd), ref["ids"], ref["w"], cfg.n_experts,
                            cfg.n_shared, tok_idx=idx)
    check_output(got["y"][idx], yref, "bf16")


# ------------------------------------------------------------------ shared expert beside the scatter kernel, under capture
def test_shared_expert_pairs_under_graph_capture():
    """With a shared expert and enough rows for the CTA-pair kernels, the shared expert's gate/up pairs run on the
    library's second stream beside the scatter kernel, and the odd-tile passes fork there a second time. The same
    call captured into a CUDA graph (both forks and joins become graph edges) and replayed gives the bits of the
    plain stream call; outputs against the oracle on a token sample."""
    case = Case(small_bf16(n_shared=1, prefill_tokens=3001, hidden=256, inter=384, logits="normal"), std=0.1)
    cfg, ex, dev = case.cfg, case.ex, case.dev
    T, Kp = case.T, 2
    ref = case.run_prefill(Kp, with_meta=False)["y"]
    ws = case.workspace(T, Kp)
    y = torch.full((T, cfg.hidden), float("nan"), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        ex.exfold_moe_prefill(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, Kp, y, ws,
                              stream=stream)   # warm-up outside the capture: the second stream is created here
        stream.synchronize()
        y.fill_(float("nan"))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ex.exfold_moe_prefill(case.layer, case.d_x, case.d_lg, case.d_wg, case.d_wu, case.d_wd, case.tables, Kp, y,
                                  ws, stream=stream)
        for _ in range(3):
            graph.replay()
        stream.synchronize()
        assert ex.exfold_device_status(ws, stream) == 0
    got = y.float().cpu().numpy()
    assert np.array_equal(got, ref)
    idx = sample_tokens(T, 40)
    check_output(got[idx], case.oracle_prefill(Kp, tok_idx=idx)["y"], "bf16")


# ------------------------------------------------------------------ decode work lists: every slicing of the gate/up kernel
@pytest.mark.parametrize("N,K,B,M,inter", [
    (64, 4, 64, 30, 384),    # 30 x 3 full slices < one round, too many to halve, 96 | I: 96-wide slices (120 items)
    (64, 4, 64, 20, 384),    # 60 full slices: the whole round is cut into halves
    (64, 4, 64, 30, 448),    # I = 3 x 128 + 64: full slices plus a natural half per expert
    (128, 8, 128, 64, 384),  # more than one round: full slices, the last partial round in halves
])
def test_decode_slicing_variants(N, K, B, M, inter):
    """The gate/up kernel deals (pool expert, slice of I) items over the SMs in several ways depending on how many there
    are (full 128-wide slices, halves, 96-wide slices, a fixed number of CTAs): each against the oracle, with the pool
    and the remapped slots bit-exact."""
    case = Case(small_bf16(n_experts=N, top_k=K, decode_batch=B, inter=inter, hidden=256, logits="normal"), std=0.1)
    got, ref = case.run_decode(M), case.oracle_decode(M)
    check_decode_meta(got, ref, M)
    check_output(got["y"], ref["y"], "bf16")


def test_chunked_host_prefill_with_a_shared_expert():
    """A host-buffer prefill call long enough to run in chunks, on a layer with a shared expert: every chunk forks
    the second stream twice (the shared expert's gate/up pairs beside the scatter kernel, then the odd-tile passes)
    while the copy streams bring the next chunk in and the previous one out. Same bits as the call on device buffers."""
    cfg = small_bf16(prefill_tokens=8500, n_experts=8, n_shared=1, hidden=128, inter=128, top_k=2, logits="normal")
    case = Case(cfg)
    ex, T, K, Kp = case.ex, case.T, cfg.top_k, 1
    ref = case.run_prefill(Kp, with_meta=False)["y"]
    ws = ex.alloc_workspace(case.layer, T, K, host_staging=True)
    ws.fill_(0xFF)
    xh, lh = case.x.pin_memory(), case.lg.pin_memory()
    for _ in range(2):
        yh = torch.full((T, cfg.hidden), float("nan"), dtype=torch.bfloat16).pin_memory()
        ex.exfold_moe_prefill_host(case.layer, xh, lh, case.d_wg, case.d_wu, case.d_wd, case.tables, Kp, yh, ws)
        assert ex.exfold_device_status(ws) == 0
        assert np.array_equal(yh.float().numpy(), ref)
    idx = sample_tokens(T, 40)
    check_output(ref[idx], case.oracle_prefill(Kp, tok_idx=idx)["y"], "bf16")
