"""Pins for the CPU oracle: it is checked against things other than itself.

* attention (alpha, o): torch's fp64 scaled-dot-product attention with an explicit mask and the KV
  heads repeated for the group;
* CAOTE score: leave-one-out recomputation of the attention output (Theorem 3.2) with torch, on every
  token of the tiny fp32 configuration and on random tiny cases; for general weights, deletion and
  renormalisation of the weights (Theorem 3.1);
* closed forms (q = 0, n = 2), invariances, the H2O mass theorem (Appendix D.1), chunking invariance;
* the FLOP model of Appendix C re-derived against the ratios the paper prints (tests/golden);
* selection against a tuple sort, compaction against multiset preservation.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2504_14051_b200 import workloads as wl


def rand_case(seed, B, Hq, Hkv, d, n, m=1, cap=None, dtype=np.float32):
    rng = np.random.default_rng(seed)
    cap = cap or n
    q = rng.standard_normal((B, Hq, m, d)).astype(dtype)
    K = rng.standard_normal((B, Hkv, cap, d)).astype(dtype)
    V = rng.standard_normal((B, Hkv, cap, d)).astype(dtype)
    lens = np.full((B,), n, dtype=np.int32)
    return q, K, V, lens


def sdpa_reference(q, K, V, lens, scale, m):
    """o [B,Hq,m,d] and alpha [B,Hq,m,cap] from torch SDPA / softmax in fp64."""
    B, Hq, _, d = q.shape
    Hkv, cap = K.shape[1], K.shape[2]
    G = Hq // Hkv
    qt = torch.from_numpy(q.astype(np.float64))
    Kt = torch.from_numpy(K.astype(np.float64)).repeat_interleave(G, dim=1)
    Vt = torch.from_numpy(V.astype(np.float64)).repeat_interleave(G, dim=1)
    mask = torch.zeros((B, 1, m, cap), dtype=torch.bool)
    for b in range(B):
        n = int(lens[b])
        for i in range(m):
            mask[b, 0, i, : n - m + i + 1] = True
    o = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt, attn_mask=mask, scale=scale)
    logits = (qt @ Kt.transpose(-1, -2)) * scale
    alpha = torch.softmax(logits.masked_fill(~mask, float("-inf")), dim=-1)
    return o.numpy(), alpha.numpy()


# ---------------------------------------------------------------- attention against torch SDPA
@pytest.mark.parametrize("B,Hq,Hkv,d,n,m,cap", [(2, 4, 2, 16, 37, 1, 40), (1, 6, 2, 8, 23, 5, 23),
                                                (1, 3, 3, 4, 9, 9, 12)])
def test_attention_matches_sdpa(B, Hq, Hkv, d, n, m, cap):
    q, K, V, lens = rand_case(7, B, Hq, Hkv, d, n, m, cap)
    lens[-1] = n - 2 if n - 2 >= m else n  # ragged
    scale = 0.37
    r = oracle.score(q, K, V, lens, scale=scale, n_new=m, base_mode="chunk_sum")
    o_ref, alpha = sdpa_reference(q, K, V, lens, scale, m)
    np.testing.assert_allclose(r["o"], o_ref, rtol=1e-12, atol=1e-14)
    # chunk-sum weights are the column sums of alpha over rows and group heads, normalised
    G = Hq // Hkv
    for b in range(B):
        nb = int(lens[b])
        for h in range(Hkv):
            hsum = alpha[b, h * G:(h + 1) * G, :, :nb].sum(axis=(0, 1))
            np.testing.assert_allclose(r["w"][b, h, :nb], hsum / (G * m), rtol=1e-12, atol=1e-15)
            assert np.isnan(r["scores"][b, h, nb:]).all()


def test_last_query_weights_use_only_last_row():
    q, K, V, lens = rand_case(11, 1, 4, 2, 8, 19, 4)
    r = oracle.score(q, K, V, lens, scale=0.5, n_new=4, base_mode="last_query")
    _, alpha = sdpa_reference(q, K, V, lens, 0.5, 4)
    for h in range(2):
        hsum = alpha[0, 2 * h:2 * h + 2, -1, :19].sum(axis=0)
        np.testing.assert_allclose(r["w"][0, h, :19], hsum / 2, rtol=1e-12)


# ---------------------------------------------------------------- Theorem 3.2: leave-one-out
def leave_one_out_errors(q1, K1, V1, scale):
    """|| o - o_{-j} ||_2 for every j: single head, single query, recomputed with torch in fp64."""
    qt = torch.from_numpy(q1.astype(np.float64))
    Kt = torch.from_numpy(K1.astype(np.float64))
    Vt = torch.from_numpy(V1.astype(np.float64))
    n = Kt.shape[0]
    full = torch.softmax((Kt @ qt) * scale, dim=0) @ Vt
    errs = np.zeros(n)
    for j in range(n):
        keep = [t for t in range(n) if t != j]
        oj = torch.softmax((Kt[keep] @ qt) * scale, dim=0) @ Vt[keep]
        errs[j] = torch.linalg.vector_norm(full - oj).item()
    return errs


@pytest.mark.parametrize("n,d", [(2, 1), (3, 4), (5, 64), (17, 4), (17, 64)])
def test_score_equals_leave_one_out_error_tiny(n, d):
    q, K, V, lens = rand_case(100 + n * d, 1, 1, 1, d, n)
    scale = 1.0 / math.sqrt(d)
    r = oracle.score(q, K, V, lens, scale=scale)
    errs = leave_one_out_errors(q[0, 0, 0], K[0, 0], V[0, 0], scale)
    np.testing.assert_allclose(r["scores"][0, 0, :n], errs, rtol=1e-9, atol=1e-13)


def test_score_equals_leave_one_out_error_every_token_of_c1():
    """Every token of the tiny fp32 configuration, each of its 4 query heads taken alone (G = 1)."""
    w = wl.WORKLOADS["c1"]
    K0, V0 = wl.initial_cache(w, "cpu")
    q, kn, vn = wl.step_inputs(w, "cpu", 0)
    n = w.init_len + 1
    K0[:, :, n - 1] = kn[:, :, 0]
    V0[:, :, n - 1] = vn[:, :, 0]
    G = w.group
    for hq in range(w.n_q_heads):
        h = hq // G
        q1 = q[:, hq:hq + 1].numpy()
        K1, V1 = K0[:, h:h + 1].numpy(), V0[:, h:h + 1].numpy()
        r = oracle.score(q1, K1, V1, np.array([n], dtype=np.int32), scale=w.scale)
        errs = leave_one_out_errors(q1[0, 0, 0], K1[0, 0, :n], V1[0, 0, :n], w.scale)
        np.testing.assert_allclose(r["scores"][0, 0, :n], errs, rtol=1e-9, atol=1e-13)
        assert (r["scores"][0, 0, :n] >= 0).all()


# ---------------------------------------------------------------- Theorem 3.1 with general weights
@pytest.mark.parametrize("mode", ["last_query", "chunk_sum", "external", "accum"])
def test_general_weights_deletion_identity(mode):
    B, Hq, Hkv, d, n, m = 1, 4, 2, 8, 13, 3
    q, K, V, lens = rand_case(5, B, Hq, Hkv, d, n, m)
    rng = np.random.default_rng(3)
    base = rng.random((B, Hkv, n)) * 3.0 if mode in ("external", "accum") else None
    r = oracle.score(q, K, V, lens, scale=0.4, n_new=m, base_mode=mode, base=base)
    for h in range(Hkv):
        w = r["w"][0, h, :n]
        assert abs(w.sum() - 1.0) < 1e-12
        Vh = V[0, h, :n].astype(np.float64)
        X = w @ Vh
        np.testing.assert_allclose(r["X"][0, h], X, rtol=1e-12, atol=1e-15)
        for j in range(n):
            w2 = np.delete(w, j) / (1.0 - w[j])  # Theorem 3.1
            assert abs(w2.sum() - 1.0) < 1e-12
            Xj = w2 @ np.delete(Vh, j, axis=0)
            assert abs(np.linalg.norm(X - Xj) - r["scores"][0, h, j]) <= 1e-10 * (1 + r["scores"][0, h, j])
    if mode == "accum":
        _, alpha = sdpa_reference(q, K, V, lens, 0.4, m)
        G = Hq // Hkv
        for h in range(Hkv):
            added = alpha[0, h * G:(h + 1) * G, :, :n].sum(axis=(0, 1))
            np.testing.assert_allclose(r["base"][0, h, :n], base[0, h] + added, rtol=1e-12)
    if mode == "external":
        np.testing.assert_allclose(r["w"][0, :, :n], base[0] / base[0].sum(-1, keepdims=True), rtol=1e-12)


# ---------------------------------------------------------------- closed forms
def test_zero_query_uniform_weights_closed_form():
    q, K, V, lens = rand_case(21, 1, 2, 1, 6, 11)
    q[:] = 0.0
    r = oracle.score(q, K, V, lens, scale=1.0)
    Vd = V[0, 0].astype(np.float64)
    expect = np.linalg.norm(Vd - Vd.mean(0), axis=1) / (11 - 1)
    np.testing.assert_allclose(r["scores"][0, 0], expect, rtol=1e-12)
    np.testing.assert_allclose(r["w"][0, 0], 1.0 / 11, rtol=1e-13)


def test_two_tokens_closed_form():
    q, K, V, lens = rand_case(22, 1, 1, 1, 5, 2)
    r = oracle.score(q, K, V, lens, scale=0.7)
    s = (K[0, 0].astype(np.float64) @ q[0, 0, 0].astype(np.float64)) * 0.7
    a = np.exp(s - s.max())
    a /= a.sum()
    dist = np.linalg.norm(V[0, 0, 0].astype(np.float64) - V[0, 0, 1].astype(np.float64))
    np.testing.assert_allclose(r["scores"][0, 0], a * dist, rtol=1e-12)


def test_single_token_and_dominant_token():
    q, K, V, lens = rand_case(23, 1, 1, 1, 4, 1)
    r = oracle.score(q, K, V, lens, scale=1.0)
    assert np.isposinf(r["scores"][0, 0, 0])
    # a token that holds almost all the weight (1 - w ~ 1e-7 here) keeps a finite, accurate score: the
    # complement is summed from the other weights, and X - v_j still has ~9 digits left in double
    q, K, V, lens = rand_case(24, 1, 1, 1, 4, 6)
    K[0, 0, 2] = q[0, 0, 0] * 4.0
    r = oracle.score(q, K, V, lens, scale=1.0)
    errs = leave_one_out_errors(q[0, 0, 0], K[0, 0], V[0, 0], 1.0)
    assert np.isfinite(r["scores"]).all() and not np.isnan(r["scores"]).any()
    assert 1e-9 < 1.0 - r["w"][0, 0, 2] < 1e-4
    np.testing.assert_allclose(r["scores"][0, 0, 2], errs[2], rtol=1e-6)


def test_external_all_zero_base_gives_zero_scores():
    q, K, V, lens = rand_case(25, 1, 1, 1, 4, 6)
    r = oracle.score(q, K, V, lens, scale=1.0, base_mode="external", base=np.zeros((1, 1, 6)))
    assert (r["scores"][0, 0] == 0).all()


# ---------------------------------------------------------------- invariants
def test_invariants():
    B, Hq, Hkv, d, n = 1, 4, 2, 8, 15
    q, K, V, lens = rand_case(31, B, Hq, Hkv, d, n)
    r0 = oracle.score(q, K, V, lens, scale=0.3)
    c0 = r0["scores"]
    assert (c0 >= 0).all()
    # all values equal -> every score is 0; a token with v_j = X scores 0
    V1 = np.broadcast_to(V[:, :, :1], V.shape).copy()
    assert np.abs(oracle.score(q, K, V1, lens, scale=0.3)["scores"]).max() < 1e-15
    V2 = V.copy()
    Xapprox = r0["X"][0, 0]
    for _ in range(60):  # fixed point: v_3 := X(v_3)
        V2[0, 0, 3] = Xapprox.astype(np.float32)
        Xapprox = oracle.score(q, K, V2, lens, scale=0.3)["X"][0, 0]
    assert oracle.score(q, K, V2, lens, scale=0.3)["scores"][0, 0, 3] < 1e-6 * c0[0, 0].max()
    # adding a constant vector to all values changes nothing; scaling values scales the scores
    shift = np.arange(d, dtype=np.float32)[None, None, None, :] * 0.25
    np.testing.assert_allclose(oracle.score(q, K, V + shift, lens, scale=0.3)["scores"], c0, rtol=1e-6)
    np.testing.assert_allclose(oracle.score(q, K, V * -2.0, lens, scale=0.3)["scores"], 2 * c0, rtol=1e-12)
    # adding the same vector to every key shifts all logits of a row by a constant -> no change
    # (0.5 steps are exact in fp32 for these magnitudes only approximately -> loose tolerance)
    kshift = np.full((1, 1, 1, d), 0.5, dtype=np.float32)
    np.testing.assert_allclose(oracle.score(q, K + kshift, V, lens, scale=0.3)["scores"], c0, rtol=1e-5)
    # permuting the slots permutes the scores
    perm = np.random.default_rng(0).permutation(n)
    rp = oracle.score(q, K[:, :, perm], V[:, :, perm], lens, scale=0.3)
    np.testing.assert_allclose(rp["scores"], c0[:, :, perm], rtol=1e-10)
    # identical queries in a group -> the grouped result equals the single-head result
    qs = np.repeat(q[:, ::2], 2, axis=1)
    rg = oracle.score(qs, K, V, lens, scale=0.3)
    r1 = oracle.score(q[:, ::2], K, V, lens, scale=0.3)
    np.testing.assert_allclose(rg["scores"], r1["scores"], rtol=1e-12)


def test_sum_errors_mode_is_sum_of_single_head_scores():
    q, K, V, lens = rand_case(41, 1, 4, 2, 8, 12)
    r = oracle.score(q, K, V, lens, scale=0.3, agg_mode="sum_errors")
    for h in range(2):
        tot = np.zeros(12)
        for g in range(2):
            r1 = oracle.score(q[:, 2 * h + g:2 * h + g + 1], K[:, h:h + 1], V[:, h:h + 1], lens, scale=0.3)
            tot += r1["scores"][0, 0]
        np.testing.assert_allclose(r["scores"][0, h], tot, rtol=1e-12)


@pytest.mark.parametrize("mode", ["chunk_sum", "last_query"])
def test_sum_errors_mode_with_a_block_of_queries_is_theorem_3_2_row_by_row(mode):
    """m > 1: every counted row i of every group head sees the first n - m + i + 1 slots; its contribution
    is the single-head, single-query score (itself pinned by leave-one-out) on the cache cut to those
    slots, and tokens the row cannot see get nothing from it."""
    B, Hq, Hkv, d, n, m, cap = 2, 6, 2, 8, 14, 4, 16
    q, K, V, lens = rand_case(43, B, Hq, Hkv, d, n, m, cap)
    lens[1] = 9
    G = Hq // Hkv
    r = oracle.score(q, K, V, lens, scale=0.3, n_new=m, base_mode=mode, agg_mode="sum_errors")
    for b in range(B):
        nb = int(lens[b])
        for h in range(Hkv):
            tot = np.zeros(nb)
            for g in range(G):
                for i in (range(m) if mode == "chunk_sum" else [m - 1]):
                    n_vis = nb - m + i + 1
                    q1 = q[b:b + 1, h * G + g:h * G + g + 1, i:i + 1]
                    r1 = oracle.score(q1, K[b:b + 1, h:h + 1, :n_vis], V[b:b + 1, h:h + 1, :n_vis],
                                      np.array([n_vis], dtype=np.int32), scale=0.3)
                    tot[:n_vis] += r1["scores"][0, 0, :n_vis]
                    # and that single-row score is the leave-one-out error of that row (Theorem 3.2)
                    errs = leave_one_out_errors(q1[0, 0, 0], K[b, h, :n_vis], V[b, h, :n_vis], 0.3)
                    np.testing.assert_allclose(r1["scores"][0, 0, :n_vis], errs, rtol=1e-9, atol=1e-13)
            np.testing.assert_allclose(r["scores"][b, h, :nb], tot, rtol=1e-12)
            assert np.isnan(r["scores"][b, h, nb:]).all()


# ---------------------------------------------------------------- H2O mass theorem, chunking
def run_accum(q_all, K, V, chunks, scale):
    """Feed T tokens causally in the given chunk sizes with no eviction; return accumulated base."""
    B, Hq, T, d = q_all.shape
    Hkv = K.shape[1]
    base = np.zeros((B, Hkv, T))
    t = 0
    for m in chunks:
        lens = np.full((B,), t + m, dtype=np.int32)
        r = oracle.score(q_all[:, :, t:t + m], K, V, lens, scale=scale, n_new=m, base_mode="accum", base=base)
        base = r["base"]
        t += m
    return base


def test_h2o_mass_theorem_and_chunking_invariance():
    B, Hq, Hkv, d, T = 1, 4, 2, 8, 24
    rng = np.random.default_rng(51)
    q_all = rng.standard_normal((B, Hq, T, d)).astype(np.float32)
    K = rng.standard_normal((B, Hkv, T, d)).astype(np.float32)
    V = rng.standard_normal((B, Hkv, T, d)).astype(np.float32)
    base_a = run_accum(q_all, K, V, [1] * T, 0.3)
    base_b = run_accum(q_all, K, V, [5, 7, 1, 11], 0.3)
    base_c = run_accum(q_all, K, V, [T], 0.3)
    G = Hq // Hkv
    np.testing.assert_allclose(base_a.sum(-1), G * T, rtol=1e-12)  # Appendix D.1: sum_j h_j = b + 1 per head
    np.testing.assert_allclose(base_a, base_b, rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(base_a, base_c, rtol=1e-11, atol=1e-14)
    # the first token attends only to itself: it received 1 from its own row at least
    assert (base_a[:, :, 0] >= G).all()


# ---------------------------------------------------------------- FastCAOTE and joint scores
def test_fast_and_joint_scores():
    q, K, V, lens = rand_case(61, 1, 1, 1, 6, 9)
    r = oracle.score(q, K, V, lens, scale=0.5)
    w, Vh = r["w"][0, 0], V[0, 0]
    # joint score of a single token is the CAOTE score
    for j in range(9):
        assert abs(oracle.joint_score(w, Vh, [j]) - r["scores"][0, 0, j]) < 1e-12
    # joint score of a pair = brute-force error of deleting both and renormalising (Appendix B)
    Vd = Vh.astype(np.float64)
    X = w @ Vd
    for a, b in itertools.combinations(range(9), 2):
        keep = [t for t in range(9) if t not in (a, b)]
        X2 = (w[keep] / w[keep].sum()) @ Vd[keep]
        assert abs(oracle.joint_score(w, Vh, [a, b]) - np.linalg.norm(X - X2)) < 1e-11
    # FastCAOTE with uniform weights coincides with CAOTE (then X is the mean of the values)
    q0 = np.zeros_like(q)
    r0 = oracle.score(q0, K, V, lens, scale=0.5)
    np.testing.assert_allclose(oracle.fast_scores(r0["w"][0, 0], Vh), r0["scores"][0, 0], rtol=1e-12)
    f = oracle.fast_scores(w, Vh)
    expect = w / (1 - w) * np.linalg.norm(Vd.mean(0) - Vd, axis=1)
    np.testing.assert_allclose(f, expect, rtol=1e-12)


@pytest.mark.parametrize("mode,G,m", [("last_query", 1, 1), ("last_query", 3, 1), ("chunk_sum", 2, 3)])
def test_fast_scores_keep_the_caote_weights_and_only_swap_the_reference_vector(mode, G, m):
    """Sec. 3.3 changes one thing: X_attn becomes the mean of the cached values. So under non-uniform
    weights the ratio FastCAOTE / CAOTE of a token must be ||mean(v) - v_j|| / ||X - v_j||, with X and the
    CAOTE score taken from oracle.score (both pinned by leave-one-out above). A wrong weight factor, a
    norm of the wrong vector or a mean over the wrong rows breaks the ratio."""
    n, d, cap = 13, 6, 16
    q, K, V, lens = rand_case(67 + G, 1, G, 1, d, n, m, cap)
    r = oracle.score(q, K, V, lens, scale=0.8, n_new=m, base_mode=mode)
    w, c, X = r["w"][0, 0, :n], r["scores"][0, 0, :n], r["X"][0, 0]
    assert w.max() / w.min() > 5.0  # far from uniform
    Vd = V[0, 0, :n].astype(np.float64)
    f = oracle.fast_scores(w, V[0, 0, :n])
    mean = torch.from_numpy(Vd).mean(dim=0).numpy()
    ratio = np.linalg.norm(mean - Vd, axis=1) / np.linalg.norm(X - Vd, axis=1)
    np.testing.assert_allclose(f / c, ratio, rtol=1e-10)
    # rows behind the length must not enter the mean
    V2 = V.copy()
    V2[0, 0, n:] = 1e6
    np.testing.assert_allclose(oracle.fast_scores(w, V2[0, 0, :n]), f, rtol=0, atol=0)


# ---------------------------------------------------------------- greedy multi-token eviction (Appendix B)
def brute_output(w, Vd, keep):
    """Attention output over the kept tokens with their weights renormalised (Theorem 3.1)."""
    return (w[keep] / w[keep].sum()) @ Vd[keep]


@pytest.mark.parametrize("n,d,k,seed", [(6, 3, 2, 1), (8, 4, 2, 2), (8, 4, 5, 3), (19, 16, 18, 4), (33, 8, 12, 5)])
def test_greedy_eviction_sequence(n, d, k, seed):
    rng = np.random.default_rng(seed)
    V = rng.standard_normal((n, d)).astype(np.float32)
    w = rng.random(n) ** 3 + 1e-3
    w /= w.sum()
    Vd = V.astype(np.float64)
    order, step, cum = oracle.greedy_evict(w, V, k)
    assert len(set(order.tolist())) == k
    X0 = w @ Vd
    present = np.ones(n, dtype=bool)
    Xprev = X0
    for t in range(k):
        # (i) the pick is the arg-min of the leave-one-out errors of the tokens still present, each
        #     recomputed from scratch (delete, renormalise, recompute the output)
        idx = np.flatnonzero(present)
        errs = []
        for j in idx:
            keep = idx[idx != j]
            errs.append(np.linalg.norm(brute_output(w, Vd, idx) - brute_output(w, Vd, keep)))
        errs = np.array(errs)
        assert idx[np.argmin(errs)] == order[t]
        np.testing.assert_allclose(step[t], errs.min(), rtol=1e-9, atol=1e-14)
        # (ii) after the pick the carried output equals sum w v over the survivors recomputed from scratch
        present[order[t]] = False
        Xnow = brute_output(w, Vd, np.flatnonzero(present))
        np.testing.assert_allclose(step[t], np.linalg.norm(Xprev - Xnow), rtol=1e-9, atol=1e-14)
        # (iii) the cumulative error is the closed-form joint score of the evicted set
        np.testing.assert_allclose(cum[t], np.linalg.norm(X0 - Xnow), rtol=1e-9, atol=1e-14)
        np.testing.assert_allclose(cum[t], oracle.joint_score(w, V, order[:t + 1]), rtol=1e-9, atol=1e-14)
        Xprev = Xnow
    # k = 1 is the plain arg-min of the CAOTE scores; k = 0 evicts nothing
    o1, s1, _ = oracle.greedy_evict(w, V, 1)
    c = w / (1 - w) * np.linalg.norm(X0 - Vd, axis=1)
    assert o1[0] == np.argmin(c) and abs(s1[0] - c.min()) < 1e-12
    assert len(oracle.greedy_evict(w, V, 0)[0]) == 0
    with pytest.raises(ValueError):
        oracle.greedy_evict(w, V, n)


def test_greedy_eviction_ties_and_pair_optimality_report():
    # equal scores: the older token (smaller pos) goes first
    V = np.array([[1.0, 0.0], [-1.0, 0.0], [0.0, 1.0], [0.0, -1.0]], dtype=np.float32)
    w = np.full(4, 0.25)
    assert oracle.greedy_evict(w, V, 1, pos=[7, 3, 9, 5])[0].tolist() == [1]
    assert oracle.greedy_evict(w, V, 1)[0].tolist() == [0]
    # greedy is a heuristic: against exhaustive search over pairs it is never better, and on random
    # inputs it is optimal about half of the time (counted, not asserted beyond "never better")
    hits = 0
    for seed in range(40):
        rng = np.random.default_rng(1000 + seed)
        n, d = 8, 3
        Vr = rng.standard_normal((n, d)).astype(np.float32)
        wr = rng.random(n) + 0.05
        wr /= wr.sum()
        order, _, cum = oracle.greedy_evict(wr, Vr, 2)
        best = min(oracle.joint_score(wr, Vr, list(pair)) for pair in itertools.combinations(range(n), 2))
        assert cum[1] >= best - 1e-12
        hits += abs(cum[1] - best) < 1e-12
    assert hits > 0


# ---------------------------------------------------------------- the paper's printed numbers
def test_post_evict_output_is_attention_over_the_retained_tokens():
    """Pins: (1) torch fp64 scaled-dot-product attention on the retained keys with the causal-in-block mask;
    (2) the correction formula of Sec. 3.1, o' = (o - sum alpha_e v_e) / (1 - sum alpha_e), built from the
    pre-eviction output and weights that oracle.score returns for one head and one query; (3) evicting
    nothing gives the pre-eviction output back."""
    rng = np.random.default_rng(31)
    B, Hq, Hkv, d, cap, m = 2, 4, 2, 16, 40, 3
    lens = np.array([37, 12], dtype=np.int32)
    q = rng.standard_normal((B, Hq, m, d)).astype(np.float32)
    K = rng.standard_normal((B, Hkv, cap, d)).astype(np.float32)
    V = rng.standard_normal((B, Hkv, cap, d)).astype(np.float32)
    scale = d ** -0.5
    evict = [[np.array([0, 5, 35, 36]), np.array([7])], [np.array([10, 11]), np.array([], dtype=np.int64)]]
    got = oracle.post_evict_output(q, K, V, lens, evict, scale=scale, n_new=m)
    G = Hq // Hkv
    for b in range(B):
        n = int(lens[b])
        for h in range(Hkv):
            keep = np.setdiff1d(np.arange(n), evict[b][h])
            kt = torch.from_numpy(K[b, h, keep]).double()[None, None]
            vt = torch.from_numpy(V[b, h, keep]).double()[None, None]
            mask = torch.from_numpy(keep[None, :] <= (n - m + np.arange(m))[:, None])  # [m, kept]
            for g in range(G):
                qt = torch.from_numpy(q[b, h * G + g]).double()[None, None]
                ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask[None, None], scale=scale)
                np.testing.assert_allclose(got[b, h * G + g], ref[0, 0].numpy(), rtol=1e-12, atol=1e-13)
    none = [[np.array([], dtype=np.int64)] * Hkv for _ in range(B)]
    r = oracle.score(q, K, V, lens, scale=scale, n_new=m, base_mode="chunk_sum")
    np.testing.assert_allclose(oracle.post_evict_output(q, K, V, lens, none, scale=scale, n_new=m), r["o"], rtol=1e-12, atol=1e-13)
    # one head, one query: w of oracle.score is that query's attention row
    q1, n1 = q[:1, :1, :1], np.array([37], dtype=np.int32)
    r1 = oracle.score(q1, K[:1, :1], V[:1, :1], n1, scale=scale, n_new=1, base_mode="last_query")
    E = np.array([3, 8, 20])
    a = r1["w"][0, 0, E]
    want = (r1["o"][0, 0, 0] - a @ V[0, 0, E].astype(np.float64)) / (1.0 - a.sum())
    got1 = oracle.post_evict_output(q1, K[:1, :1], V[:1, :1], n1, [[E]], scale=scale, n_new=1)
    np.testing.assert_allclose(got1[0, 0, 0], want, rtol=1e-11, atol=1e-13)


def test_flop_model_matches_printed_ratios():
    """Appendix C: the FLOP formulas with Llama-3.1-8B dimensions reproduce the printed ratio tables."""
    path = os.path.join(os.path.dirname(__file__), "golden", "appendix_c_flop_ratios.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    L, d, d_kv, d_ffn, d_v = 32, 4096, 1024, 14336, 128256
    for phase, s, r_caote, r_fast in rows:
        s = int(s)
        per_tok = 2 * L * d * (d + d_kv + d_ffn + 2 * s + 6)
        model = per_tok * s + d * d_v if phase == "prefill" else per_tok + d * d_v
        caote = L * s * (7 * d + 3)
        fast = L * s * (4 * d + 3) + L
        if phase == "prefill":
            # the printed prefill ratios are only reproduced to within a factor ~2 by the printed
            # formulas (they fall as 1/s in the table but not in the formulas); check the order of
            # magnitude and the CAOTE : FastCAOTE proportion, which is what the formulas fix
            assert 0.2 < (caote / model) / float(r_caote) < 5.0
            assert abs((fast / caote) - float(r_fast) / float(r_caote)) < 0.03
        else:
            assert abs(caote / model - float(r_caote)) < 0.006
            assert abs(fast / model - float(r_fast)) < 0.003


# ---------------------------------------------------------------- selection and compaction
def test_select_matches_tuple_sort_and_edge_cases():
    rng = np.random.default_rng(71)
    B, Hkv, cap = 3, 2, 20
    scores = rng.random((B, Hkv, cap)).round(1)  # many ties
    pos = np.stack([np.stack([rng.permutation(cap) for _ in range(Hkv)]) for _ in range(B)])
    lens = np.array([20, 13, 7])
    budget = np.array([20, 1, 4])  # k = 0, n - 1, 3
    ev, k = oracle.select_evict(scores, lens, budget, pos)
    assert k.tolist() == [0, 12, 3]
    for b in range(B):
        for h in range(Hkv):
            n = lens[b]
            order = sorted(range(n), key=lambda j: (scores[b, h, j], pos[b, h, j]))
            assert sorted(order[:k[b]]) == ev[b][h].tolist()
    # all-equal scores: the oldest tokens go first
    ev, k = oracle.select_evict(np.ones((1, 1, 6)), [6], [4], np.array([[[5, 0, 3, 1, 4, 2]]]))
    assert ev[0][0].tolist() == [1, 3]
    ev, _ = oracle.select_evict(np.ones((1, 1, 6)), [6], [4], None)
    assert ev[0][0].tolist() == [0, 1]


def test_compact_preserves_survivors():
    rng = np.random.default_rng(81)
    B, Hkv, cap, d = 2, 2, 12, 3
    K = rng.standard_normal((B, Hkv, cap, d))
    pos = np.tile(np.arange(cap), (B, Hkv, 1))
    lens = np.array([12, 9])
    scores = rng.random((B, Hkv, cap))
    ev, k = oracle.select_evict(scores, lens, [8, 9], pos)
    (K2, pos2), lens2 = oracle.compact([K, pos], lens, ev)
    assert lens2.tolist() == [8, 9]
    for b in range(B):
        for h in range(Hkv):
            keep = [j for j in range(lens[b]) if j not in set(ev[b][h].tolist())]
            assert pos2[b, h, :lens2[b]].tolist() == keep
            np.testing.assert_array_equal(K2[b, h, :lens2[b]], K[b, h, keep])
