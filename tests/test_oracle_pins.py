"""Pins for the CPU oracle: every check here compares it with something other than itself
(a library routine, a closed form, brute force, an invariant the equations imply)."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si


def tiny_layer(seed=1, N=6, d=16, I=24, T=10, n_shared=0, dtype="f32", logits="normal"):
    cfg = si.LayerConfig("t", N, n_shared, d, I, 2, dtype, T, (1,), 4, (2,), seed=seed, logits=logits)
    x = si.hidden_states(cfg, T)
    lg = si.router_logits(cfg, T)
    wg, wu, wd = si.expert_weights(cfg, std=0.3)
    return cfg, x, lg, wg, wu, wd


def rand_tables(N, seed=0, unobs=0.0):
    g = np.random.default_rng(seed)
    S = g.uniform(-2, 2, (N, N)).astype(np.float32)
    L = g.uniform(0.05, 1, (N, N)).astype(np.float32)
    if unobs:
        m = g.uniform(size=(N, N)) < unobs
        S[m], L[m] = 0.0, 1e30
    np.fill_diagonal(S, 1)
    np.fill_diagonal(L, 0)
    h = np.exp(g.uniform(0, np.log(3.2), N)).astype(np.float32)
    lnh = np.log(h.astype(np.float64)).astype(np.float32)
    return S, L, h, lnh


def A(t):
    return si.as_oracle_array(t)


def torch_unfolded(x, lg, wg, wu, wd, K, N, n_shared):
    """Textbook SwiGLU-MoE with library ops in fp64 (Eq. 1-3)."""
    x, wg, wu, wd = (t.to(torch.float64) for t in (x, wg, wu, wd))
    top = torch.topk(lg.to(torch.float64), K, dim=1)
    w = torch.softmax(top.values, dim=1)
    y = torch.zeros_like(x)
    for i in range(x.shape[0]):
        for k in range(K):
            e = int(top.indices[i, k])
            a = torch.nn.functional.silu(wg[e] @ x[i]) * (wu[e] @ x[i])
            y[i] += w[i, k] * (wd[e] @ a)
        for s in range(n_shared):
            e = N + s
            y[i] += wd[e] @ (torch.nn.functional.silu(wg[e] @ x[i]) * (wu[e] @ x[i]))
    return y.numpy(), top.indices.numpy(), w.numpy()


@pytest.mark.parametrize("dtype,n_shared", [("f32", 0), ("bf16", 0), ("f32", 1)])
def test_unfolded_layer_matches_library(dtype, n_shared):
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=3, N=6, T=12, n_shared=n_shared, dtype=dtype)
    K = 3
    ids, w, w64 = oracle.gate(lg.numpy(), K)
    y = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), ids, w, 6, n_shared)
    yr, ir, wr = torch_unfolded(x, lg, wg, wu, wd, K, 6, n_shared)
    assert np.array_equal(ids, ir)
    np.testing.assert_allclose(w64, wr, rtol=1e-12)
    np.testing.assert_allclose(w, wr, rtol=1e-6)
    np.testing.assert_allclose(y, yr, rtol=2e-6, atol=2e-6 * np.abs(yr).max())


def test_gate_ties_take_lower_id_and_weights_sum_to_one():
    lg = np.zeros((2, 5), np.float32)
    lg[1] = [1, 3, 3, 0, 3]
    ids, w, w64 = oracle.gate(lg, 3)
    assert ids[0].tolist() == [0, 1, 2]
    assert ids[1].tolist() == [1, 2, 4]
    np.testing.assert_allclose(w64.sum(1), 1.0, rtol=1e-14)
    np.testing.assert_allclose(w64[1], 1 / 3, rtol=1e-14)


def test_full_budget_reproduces_unfolded():
    """K' = K: no route is omitted, Eq. 13 is the identity, Eq. 4 equals Eq. 3."""
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=5, N=8, T=16)
    K = 4
    S, L, h, lnh = rand_tables(8, 1)
    ids, w, _ = oracle.gate(lg.numpy(), K)
    y0 = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), ids, w, 8)
    # with h == 1 the ranking key is the logit: same slot order, bit-identical output
    one, zero = np.ones(8, np.float32), np.zeros(8, np.float32)
    f1 = oracle.prefill_fold(lg.numpy(), K, K, S, L, one, zero)
    assert np.array_equal(f1["ids"], ids) and np.array_equal(f1["w"], w)
    y1 = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), f1["ids"], f1["w"], 8)
    assert np.array_equal(y0, y1)
    # general h only permutes the slots
    f2 = oracle.prefill_fold(lg.numpy(), K, K, S, L, h, lnh)
    assert np.array_equal(np.sort(f2["ids"], 1), np.sort(ids, 1))
    y2 = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), f2["ids"], f2["w"], 8)
    np.testing.assert_allclose(y2, y0, rtol=1e-6, atol=1e-7)
    # decode with a pool at least as large as the union: Eq. 14 is the identity
    for M in (8, 7):
        dec = oracle.decode_fold(lg.numpy(), K, M, S, L, h)
        if dec["pool_size"] < M or M == 8:
            assert np.array_equal(dec["ids"], ids) and np.array_equal(dec["w"], w)
            assert set(dec["pool_ids"][:dec["pool_size"]].tolist()) == set(ids.reshape(-1).tolist())


@pytest.mark.parametrize("n_shared", [0, 1])
def test_metadata_form_equals_eq4_written_out(n_shared):
    """Folding the weight (Eq. 13 / 14) and then running K' experts equals running every
    term of Eq. 4 separately."""
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=7, N=8, T=14, n_shared=n_shared)
    K = 4
    S, L, h, lnh = rand_tables(8, 2, unobs=0.1)
    for Kp in (1, 2, 3):
        f = oracle.prefill_fold(lg.numpy(), K, Kp, S, L, h, lnh)
        ym = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), f["ids"], f["w"], 8, n_shared)
        y4 = oracle.prefill_eq4(A(x), lg.numpy(), A(wg), A(wu), A(wd), 8, n_shared, K, Kp, S, L, lnh)
        np.testing.assert_allclose(ym, y4, rtol=2e-6, atol=2e-6 * np.abs(y4).max())
    for M in (1, 2, 4):
        dec = oracle.decode_fold(lg.numpy(), K, M, S, L, h)
        ym = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), dec["ids"], dec["w"], 8, n_shared)
        pool = dec["pool_ids"][:dec["pool_size"]]
        y4 = oracle.decode_eq4(A(x), lg.numpy(), A(wg), A(wu), A(wd), 8, n_shared, K, pool, S, L)
        np.testing.assert_allclose(ym, y4, rtol=2e-6, atol=2e-6 * np.abs(y4).max())


def test_prefill_selection_brute_force():
    """Eq. 10: the retained set is the K'-subset of the routed experts with the largest
    sum of w*h (checked over all subsets, in double, on the literal product)."""
    g = np.random.default_rng(11)
    N, K = 10, 5
    lg = g.standard_normal((200, N)).astype(np.float32)
    S, L, h, lnh = rand_tables(N, 3)
    ids, w, w64 = oracle.gate(lg, K)
    for Kp in (1, 2, 4):
        f = oracle.prefill_fold(lg, K, Kp, S, L, h, lnh)
        assert f["mismatch"] == 0
        for i in range(lg.shape[0]):
            contrib = w64[i] * h[ids[i]].astype(np.float64)
            best = max(itertools.combinations(range(K), Kp), key=lambda c: sum(contrib[list(c)]))
            assert set(f["ids"][i].tolist()) == set(ids[i][list(best)].tolist())
            # retained routes are listed first, in descending contribution
            got = [contrib[list(ids[i]).index(e)] for e in f["ids"][i]]
            assert all(got[j] >= got[j + 1] for j in range(Kp - 1))
    # h == 1: the retained set is simply the top-K' by logit, in router order
    f = oracle.prefill_fold(lg, K, 2, S, L, np.ones(N, np.float32), np.zeros(N, np.float32))
    assert np.array_equal(f["ids"], ids[:, :2])


def test_min_loss_assignment_enumerated():
    """Eq. 12 by enumeration, including a planted unique minimum and an all-unobserved row."""
    g = np.random.default_rng(12)
    N, K, Kp = 9, 5, 2
    lg = g.standard_normal((300, N)).astype(np.float32)
    S, L, h, lnh = rand_tables(N, 4, unobs=0.15)
    L[3, :] = 1e30
    L[3, 3] = 0
    f = oracle.prefill_fold(lg, K, Kp, S, L, h, lnh)
    ids, w, w64 = oracle.gate(lg, K)
    for i in range(lg.shape[0]):
        kept = f["ids"][i].tolist()
        omitted = [e for e in ids[i].tolist() if e not in kept]
        assert sorted(f["omit_src"][i].tolist()) == sorted(omitted)
        for s, t in zip(f["omit_src"][i], f["omit_tgt"][i]):
            cands = sorted(kept)
            losses = [L[s, c] for c in cands]
            assert t == cands[int(np.argmin(losses))]  # first minimum = lower id on ties
    Lp = np.full((N, N), 0.9, np.float32)
    Lp[:, 7] = 0.01  # expert 7 is everyone's best target whenever it is retained
    f = oracle.prefill_fold(lg, K, Kp, S, Lp, h, lnh)
    has7 = (f["ids"] == 7).any(1)
    assert has7.any()
    assert (f["omit_tgt"][has7] == 7).all()


def test_fold_weight_bookkeeping():
    """Eq. 13 / 14: with S == 1 the folded weights still sum to 1; with S == 0 folding is
    plain truncation without renormalisation."""
    g = np.random.default_rng(13)
    N, K = 12, 6
    lg = g.standard_normal((64, N)).astype(np.float32)
    _, L, h, lnh = rand_tables(N, 5)
    ids, w, w64 = oracle.gate(lg, K)
    S1 = np.ones((N, N), np.float32)
    S0 = np.zeros((N, N), np.float32)
    np.fill_diagonal(S0, 1)
    for Kp in (1, 3):
        f = oracle.prefill_fold(lg, K, Kp, S1, L, h, lnh)
        np.testing.assert_allclose(f["w"].astype(np.float64).sum(1), 1.0, atol=3e-7)
        f0 = oracle.prefill_fold(lg, K, Kp, S0, L, h, lnh)
        for i in range(lg.shape[0]):
            for e, we in zip(f0["ids"][i], f0["w"][i]):
                assert we == w[i][list(ids[i]).index(e)]
    for M in (2, 5):
        d1 = oracle.decode_fold(lg, K, M, S1, L, h)
        np.testing.assert_allclose(d1["w"].astype(np.float64).sum(1), 1.0, atol=3e-7)
        d0 = oracle.decode_fold(lg, K, M, S0, L, h)
        inpool = np.isin(ids, d0["pool_ids"][:d0["pool_size"]])
        assert np.array_equal(d0["w"][inpool], w[inpool])
        assert (d0["w"][~inpool] == 0).all()


def test_decode_pool_invariants_and_listing_semantics():
    g = np.random.default_rng(14)
    N, K, B = 16, 4, 12
    lg = g.standard_normal((B, N)).astype(np.float32)
    S, L, h, lnh = rand_tables(N, 6, unobs=0.05)
    ids, w, w64 = oracle.gate(lg, K)
    union = sorted(set(ids.reshape(-1).tolist()))
    for M in (1, 3, 8, 16):
        dec = oracle.decode_fold(lg, K, M, S, L, h)
        P = dec["pool_size"]
        pool = dec["pool_ids"][:P].tolist()
        assert P == min(M, len(union)) and set(pool) <= set(union)
        assert (dec["pool_ids"][P:] == -1).all()
        # Eq. 11 in plain numpy: aggregate score, best M of the union
        score = np.zeros(N)
        for i in range(B):
            score[ids[i]] += w64[i]
        score *= h.astype(np.float64)
        np.testing.assert_allclose(dec["score"], score, rtol=1e-13)
        order = sorted(union, key=lambda e: (-score[e], e))
        assert pool == order[:P]
        mask = sum(1 << e for e in pool)
        assert int(dec["pool_mask"][0]) == mask
        # every id after the remap is in the pool; retained slots are untouched
        assert np.isin(dec["ids"], pool).all()
        kept = np.isin(ids, pool)
        assert np.array_equal(dec["ids"][kept], ids[kept]) and np.array_equal(dec["w"][kept], w[kept])
        # the per-route remapping kernel of the appendix: two table lookups and one multiply per slot
        tgt, scl = dec["target"], dec["scale"]
        assert np.array_equal(dec["ids"], tgt[ids])
        np.testing.assert_allclose(dec["w"], (w64 * scl[ids].astype(np.float64)).astype(np.float32), rtol=0)
        for s in range(N):
            if s in pool:
                assert tgt[s] == s and scl[s] == 1
            else:
                cands = sorted(pool)
                assert tgt[s] == cands[int(np.argmin([L[s, c] for c in cands]))]
                assert scl[s] == S[s, tgt[s]]


def test_prefill_safeguards():
    """Loss threshold, rescale and confidence split, each against its own definition in numpy."""
    g = np.random.default_rng(17)
    N, K, Kp = 10, 5, 2
    lg = g.standard_normal((120, N)).astype(np.float32)
    S, L, h, lnh = rand_tables(N, 9, unobs=0.1)
    base = oracle.prefill_fold(lg, K, Kp, S, L, h, lnh)
    off = oracle.prefill_fold_safe(lg, K, Kp, S, L, lnh)
    for k in ("ids", "w", "omit_src", "omit_tgt"):
        assert np.array_equal(off[k], base[k])           # all safeguards off = plain Eq. 13
    ids, w, w64 = oracle.gate(lg, K)
    thr = 0.6
    for rescale, conf in ((False, False), (True, False), (False, True), (True, True)):
        got = oracle.prefill_fold_safe(lg, K, Kp, S, L, lnh, loss_thr=thr, rescale=rescale, confidence=conf)
        assert np.array_equal(got["ids"], base["ids"]) and np.array_equal(got["omit_src"], base["omit_src"])
        for i in range(lg.shape[0]):
            kept = got["ids"][i].tolist()
            wk = {e: float(w64[i][list(ids[i]).index(e)]) for e in ids[i]}
            wt = {t: wk[t] for t in kept}
            ksum = sum(wk[t] for t in kept)
            for s, t in zip(got["omit_src"][i], got["omit_tgt"][i]):
                adm = sorted(c for c in kept if not (L[s, c] > thr))
                if not adm:
                    assert t == -1
                    continue
                assert t == adm[int(np.argmin([L[s, c] for c in adm]))]
                c = float(np.clip(1.0 - np.float64(L[s, t]), 0, 1)) if conf else 1.0
                wt[t] += wk[s] * c * float(S[s, t])
                if conf:
                    for t2 in kept:
                        wt[t2] += wk[s] * (1 - c) * wk[t2] / ksum
            if rescale and sum(wt.values()) > 0:
                f = 1.0 / sum(wt.values())                 # the K routed weights sum to 1
                wt = {t: v * f for t, v in wt.items()}
            np.testing.assert_allclose(got["w"][i], [wt[t] for t in kept], rtol=1e-6, atol=1e-7)
            if rescale and sum(wt.values()) > 0:
                np.testing.assert_allclose(got["w"][i].astype(np.float64).sum(), 1.0, atol=1e-6)
    # confidence split with S == 1: nothing is lost whatever the losses are
    S1 = np.ones((N, N), np.float32)
    got = oracle.prefill_fold_safe(lg, K, Kp, S1, L, lnh, confidence=True)
    np.testing.assert_allclose(got["w"].astype(np.float64).sum(1), 1.0, atol=1e-6)
    # threshold below every loss: every omitted route is dropped; rescaling restores the sum
    got = oracle.prefill_fold_safe(lg, K, Kp, S, L, lnh, loss_thr=-1.0, rescale=True)
    assert (got["omit_tgt"] == -1).all()
    np.testing.assert_allclose(got["w"].astype(np.float64).sum(1), 1.0, atol=1e-6)


def test_static_pool_and_listing_remap():
    """Static pool = the M experts with the largest calibration norm; per-route remap = the appendix
    listing (two table lookups, one multiply per slot); with the dynamic pool's tables the static remap
    reproduces the dynamic one; M = N is the unfolded layer."""
    g = np.random.default_rng(16)
    N, K, B = 16, 4, 20
    lg = g.standard_normal((B, N)).astype(np.float32)
    S, L, h, lnh = rand_tables(N, 8, unobs=0.05)
    h[3] = h[9]  # a tie in the norms: the lower id must win
    ids, w, w64 = oracle.gate(lg, K)
    for M in (1, 5, 16):
        sp = oracle.static_pool(M, S, L, h)
        order = sorted(range(N), key=lambda e: (-float(h[e]), e))
        assert sp["pool_ids"].tolist() == order[:M]
        pool = sorted(order[:M])
        for s in range(N):
            if s in pool:
                assert sp["target"][s] == s and sp["scale"][s] == 1
            else:
                assert sp["target"][s] == pool[int(np.argmin([L[s, c] for c in pool]))]
                assert sp["scale"][s] == S[s, sp["target"][s]]
        dec = oracle.decode_static(lg, K, sp["target"], sp["scale"])
        assert np.array_equal(dec["ids"], sp["target"][ids])
        assert np.array_equal(dec["w"], (w64 * sp["scale"][ids].astype(np.float64)).astype(np.float32))
        assert np.isin(dec["ids"], pool).all()
        if M == N:
            assert np.array_equal(dec["ids"], ids) and np.array_equal(dec["w"], w)
    dyn = oracle.decode_fold(lg, K, 5, S, L, h)
    st = oracle.decode_static(lg, K, dyn["target"], dyn["scale"])
    assert np.array_equal(st["ids"], dyn["ids"]) and np.array_equal(st["w"], dyn["w"])


def test_single_token_decode_equals_prefill():
    """B = 1: Eq. 11 reduces to Eq. 10 with K' = M, so both modes give the same output."""
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=15, N=8, T=6)
    K, M = 4, 2
    S, L, h, lnh = rand_tables(8, 7)
    for i in range(6):
        li = lg.numpy()[i:i + 1]
        dec = oracle.decode_fold(li, K, M, S, L, h)
        pre = oracle.prefill_fold(li, K, M, S, L, h, lnh)
        assert dec["pool_ids"].tolist() == pre["ids"][0].tolist()
        yd = oracle.moe_apply(A(x[i:i + 1]), A(wg), A(wu), A(wd), dec["ids"], dec["w"], 8)
        yp = oracle.moe_apply(A(x[i:i + 1]), A(wg), A(wu), A(wd), pre["ids"], pre["w"], 8)
        np.testing.assert_allclose(yd, yp, rtol=2e-6, atol=1e-7)


# ---------------- calibration (Eq. 6-9) ----------------

def test_calibration_single_token_closed_form():
    """One token, lambda = 0: s* = <v,u>/|v|^2 and loss = 1 - cos^2(u,v)."""
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=21, N=4, T=1)
    K = 2
    ids, _, _ = oracle.gate(lg.numpy(), K)
    out = oracle.expert_outputs(A(x), A(wg), A(wu), A(wd), ids)
    cal = oracle.calibrate(A(x), lg.numpy(), A(wg), A(wu), A(wd), 4, K, lam=0.0, clip_lo=-1e9,
                           clip_hi=1e9, eps=0.0)
    a, b = ids[0]
    u, v = out[0, 0], out[0, 1]
    np.testing.assert_allclose(cal["S"][a, b], u @ v / (v @ v), rtol=1e-6)
    np.testing.assert_allclose(cal["S"][b, a], u @ v / (u @ u), rtol=1e-6)
    cos2 = (u @ v) ** 2 / ((u @ u) * (v @ v))
    np.testing.assert_allclose(cal["L"][a, b], 1 - cos2, rtol=1e-5)
    np.testing.assert_allclose(cal["L"][b, a], 1 - cos2, rtol=1e-5)
    np.testing.assert_allclose(cal["h"][a], np.linalg.norm(u), rtol=1e-6)
    assert cal["n_obs"][a, b] == 1 and cal["n_obs"].sum() == 2
    assert cal["unobserved"] == 2


@pytest.mark.parametrize("mode", [0, 1])
def test_calibration_equals_weighted_least_squares(mode):
    """lambda = 0: Eq. 8 is the weighted least-squares fit of u on v (library lstsq on
    sqrt(w)-scaled stacked vectors); lambda > 0: A/(B+lambda) from independently summed A, B;
    Eq. 9 from the residuals directly (not the expanded form)."""
    N, K, m = 5, 3, 40
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=22, N=N, T=m)
    if mode == 0:
        ids, _, _ = oracle.gate(lg.numpy(), K)
    else:
        ids = np.tile(np.arange(N, dtype=np.int32), (m, 1))
    out = oracle.expert_outputs(A(x), A(wg), A(wu), A(wd), ids)
    for lam in (0.0, 1e-3):
        cal = oracle.calibrate(A(x), lg.numpy(), A(wg), A(wu), A(wd), N, K, lam=lam, clip_lo=-1e9,
                               clip_hi=1e9, eps=1e-12, mode=mode)
        for s in range(N):
            for t in range(N):
                if s == t:
                    assert cal["S"][s, t] == 1 and cal["L"][s, t] == 0
                    continue
                rows = [(i, list(ids[i]).index(s), list(ids[i]).index(t)) for i in range(m)
                        if s in ids[i] and t in ids[i]]
                assert cal["n_obs"][s, t] == len(rows)
                if not rows:
                    assert cal["S"][s, t] == 0 and cal["L"][s, t] == np.float32(1e30)
                    continue
                U = np.stack([out[i, a] for i, a, b in rows])
                V = np.stack([out[i, b] for i, a, b in rows])
                wts = np.linalg.norm(U, axis=1)  # source-output-norm weighting
                if lam == 0.0:
                    sw = np.sqrt(wts)[:, None]
                    sol = np.linalg.lstsq((sw * V).reshape(-1, 1), (sw * U).reshape(-1), rcond=None)[0][0]
                else:
                    sol = (wts * (U * V).sum(1)).sum() / ((wts * (V * V).sum(1)).sum() + lam)
                np.testing.assert_allclose(cal["S"][s, t], sol, rtol=2e-6)
                sst = float(cal["S"][s, t])
                res = (wts * ((U - sst * V) ** 2).sum(1)).sum() / ((wts * (U * U).sum(1)).sum() + 1e-12)
                np.testing.assert_allclose(cal["L"][s, t], res, rtol=1e-4, atol=1e-7)
        for e in range(N):
            norms = [np.linalg.norm(out[i, list(ids[i]).index(e)]) for i in range(m) if e in ids[i]]
            np.testing.assert_allclose(cal["h"][e], np.mean(norms), rtol=1e-6)
            np.testing.assert_allclose(cal["lnh"][e], np.log(np.float64(cal["h"][e])), rtol=1e-6, atol=1e-7)


def test_calibration_clip_and_ridge():
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=23, N=4, T=30)
    wd2 = wd.clone()
    wd2[1] = 9.0 * wd[0]
    wg2, wu2 = wg.clone(), wu.clone()
    wg2[1], wu2[1] = wg[0], wu[0]     # expert 1 == 9 x expert 0
    free = oracle.calibrate(A(x), lg.numpy(), A(wg2), A(wu2), A(wd2), 4, 2, lam=0.0, clip_lo=-1e9, clip_hi=1e9)
    clip = oracle.calibrate(A(x), lg.numpy(), A(wg2), A(wu2), A(wd2), 4, 2, lam=0.0)
    if free["n_obs"][1, 0] > 0:
        np.testing.assert_allclose(free["S"][1, 0], 9.0, rtol=1e-6)
        assert clip["S"][1, 0] == 4.0                      # clipped to [-4, 4]
        # loss uses the clipped scalar: |9v - 4v|^2 / |9v|^2 = 25/81
        np.testing.assert_allclose(clip["L"][1, 0], 25.0 / 81.0, rtol=1e-5)
    rid = oracle.calibrate(A(x), lg.numpy(), A(wg), A(wu), A(wd), 4, 2, lam=1e-3)
    Am, Bm, Cm = rid["stats"]
    obs = rid["n_obs"] > 0
    np.testing.assert_allclose(rid["S"][obs], np.clip(Am[obs] / (Bm[obs] + 1e-3), -4, 4), rtol=1e-6)


def test_alpha_recovery():
    """An omitted expert whose output is alpha times a retained expert's output is recovered
    exactly: calibration finds S = alpha, L = 0, and folding reproduces the unfolded layer."""
    N, K, T = 4, 2, 48
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=24, N=N, T=T)
    alpha = -1.75
    wg[1], wu[1] = wg[0], wu[0]
    wd[1] = alpha * wd[0]
    lgn = lg.numpy().copy()
    lgn[:, 0] += 6.0   # expert 0 always routed first, expert 1 always second
    lgn[:, 1] += 4.0
    cal = oracle.calibrate(A(x), lgn, A(wg), A(wu), A(wd), N, K, lam=0.0)
    np.testing.assert_allclose(cal["S"][1, 0], alpha, rtol=1e-6)
    np.testing.assert_allclose(cal["S"][0, 1], 1 / alpha, rtol=1e-6)
    assert cal["L"][1, 0] < 1e-10 and cal["L"][0, 1] < 1e-10
    np.testing.assert_allclose(cal["h"][1] / cal["h"][0], abs(alpha), rtol=1e-6)
    ids, w, _ = oracle.gate(lgn, K)
    y_full = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), ids, w, N)
    h = np.array([1.0, 1e-3, 1, 1], np.float32)          # keep expert 0, fold expert 1
    f = oracle.prefill_fold(lgn, K, 1, cal["S"], cal["L"], h, np.log(h.astype(np.float64)).astype(np.float32))
    assert (f["ids"] == 0).all() and (f["omit_src"] == 1).all() and (f["omit_tgt"] == 0).all()
    y_fold = oracle.moe_apply(A(x), A(wg), A(wu), A(wd), f["ids"], f["w"], N)
    np.testing.assert_allclose(y_fold, y_full, rtol=1e-5, atol=1e-6 * np.abs(y_full).max())
    # with the paper's ridge (lambda = 1e-3) the scalar shrinks to alpha * B / (B + lambda)
    rid = oracle.calibrate(A(x), lgn, A(wg), A(wu), A(wd), N, K, lam=1e-3)
    Bm = rid["stats"][1]
    np.testing.assert_allclose(rid["S"][1, 0], alpha * Bm[1, 0] / (Bm[1, 0] + 1e-3), rtol=1e-6)


def test_sort_routes_is_stable_counting_sort():
    g = np.random.default_rng(31)
    ids = g.integers(0, 7, size=(50, 3)).astype(np.int32)
    ids[ids == 4] = 5   # an empty group
    perm, off = oracle.sort_routes(ids, 7)
    ref = np.argsort(ids.reshape(-1), kind="stable")
    assert np.array_equal(perm, ref)
    assert np.array_equal(off, np.concatenate([[0], np.cumsum(np.bincount(ids.reshape(-1), minlength=7))]))


def test_paper_constants_fixture():
    """Values the paper prints: calibration constants and the 6.00 MiB table storage."""
    import json
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")) as f:
        c = json.load(f)
    v = c["values"]
    mib = v["layers"] * v["experts"] ** 2 * 4 * v["tables_per_layer"] / 2 ** 20
    assert abs(mib - v["storage_mib"]) < 1e-9
    import inspect
    sig = inspect.signature(oracle.calibrate)
    assert sig.parameters["lam"].default == v["ridge_lambda"]
    assert sig.parameters["clip_lo"].default == v["clip"][0] and sig.parameters["clip_hi"].default == v["clip"][1]
    cfg, x, lg, wg, wu, wd = tiny_layer(seed=2, N=5, T=3)
    cal = oracle.calibrate(A(x), lg.numpy(), A(wg), A(wu), A(wd), 5, 2)
    assert (cal["L"][cal["n_obs"] == 0][~np.eye(5, dtype=bool)[cal["n_obs"] == 0]] == np.float32(v["unobserved_loss"])).all()
    assert (np.diag(cal["S"]) == v["self_scalar"]).all()


def test_oracle_regression_snapshot():
    """The oracle on the tiny seeded layer still gives the values stored by tests/golden/make_oracle_golden.py
    (a guard against accidental changes to the oracle's arithmetic, not a pin of its correctness)."""
    import importlib.util
    import json
    import os
    here = os.path.join(os.path.dirname(__file__), "golden")
    spec = importlib.util.spec_from_file_location("make_oracle_golden", os.path.join(here, "make_oracle_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.snapshot()
    with open(os.path.join(here, "oracle_tiny.json")) as f:
        ref = json.load(f)
    for k, v in ref.items():
        if isinstance(v, str):
            continue
        if isinstance(v, list) and v and isinstance(v[0], int):
            assert now[k] == v, k
        else:
            np.testing.assert_allclose(np.asarray(now[k], np.float64), np.asarray(v, np.float64), rtol=1e-6, atol=1e-9,
                                       err_msg=k)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_router_logits_against_library_matmul_and_closed_forms(dtype):
    """r = W_r x (the scores Eq. 2 ranks): equals a float64 library matmul of the same bit patterns; one-hot
    router rows read single coordinates of x (a transposed operand or a wrong stride fails this); a constant
    row e+1 against x = 1 gives d (e+1)."""
    g = torch.Generator().manual_seed(7)
    T, N, d = 13, 5, 24
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    x = torch.randn(T, d, generator=g).to(tdt)
    wr = (0.3 * torch.randn(N, d, generator=g)).to(tdt)
    r32, r64 = oracle.router_logits(A(x), A(wr))
    ref = x.to(torch.float64) @ wr.to(torch.float64).T
    np.testing.assert_allclose(r64, ref.numpy(), rtol=1e-13, atol=1e-13)
    assert np.array_equal(r32, r64.astype(np.float32))
    onehot = torch.zeros(N, d)
    cols = [3, 0, 23, 7, 11]
    for e, c in enumerate(cols):
        onehot[e, c] = 1.0
    r32, _ = oracle.router_logits(A(x), A(onehot.to(tdt)))
    assert np.array_equal(r32, x.to(torch.float32).numpy()[:, cols])
    const = (torch.arange(1, N + 1, dtype=torch.float32)[:, None] * torch.ones(N, d)).to(tdt)
    r32, _ = oracle.router_logits(A(torch.ones(T, d).to(tdt)), A(const))
    assert np.array_equal(r32, np.tile(d * np.arange(1, N + 1, dtype=np.float32), (T, 1)))
