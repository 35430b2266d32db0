"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same bits."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_14051_b200 as P
from paper_2504_14051_b200 import workloads as wl

from parity import (assert_close, check_evicted, check_scores_and_o, f32, oracle_for, sub_problem)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_case(seed, B, Hq, Hkv, d, cap, m, dtype, lens):
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn((B, Hq, m, d), generator=g).to(dtype).to(DEV)
    K = torch.randn((B, Hkv, cap, d), generator=g).to(dtype).to(DEV)
    V = torch.randn((B, Hkv, cap, d), generator=g).to(dtype).to(DEV)
    lens = torch.tensor(lens, dtype=torch.int32, device=DEV)
    return q, K, V, lens


def run_score(q, K, V, lens, m, mode, base=None, scale=None):
    B, Hq, _, d = q.shape
    Hkv, cap = K.shape[1], K.shape[2]
    scale = d ** -0.5 if scale is None else scale
    p = P.make_params(B, Hq, Hkv, d, cap, m, q.dtype, scale, mode)
    ws = P.alloc_workspace(p, DEV)
    o = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    scores = torch.full((B, Hkv, cap), -7.0, dtype=torch.float32, device=DEV)
    P.caote_score(p, q, K, V, lens, base, o, scores, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    return p, ws, o, scores


SHAPES = [
    # B, Hq, Hkv, d, cap, m, lens
    (1, 1, 1, 64, 16, 1, [1]),
    (1, 1, 1, 64, 16, 1, [2]),
    (2, 4, 2, 64, 80, 1, [63, 80]),
    (2, 8, 2, 128, 300, 1, [257, 129]),
    (1, 7, 1, 128, 1100, 1, [1031]),
    (3, 16, 2, 128, 200, 1, [200, 0, 65]),
    (1, 14, 2, 128, 400, 3, [333]),
    (2, 8, 4, 64, 272, 128, [272, 130]),
    (1, 4, 1, 128, 520, 128, [515]),
    (1, 32, 2, 128, 96, 5, [5]),
    # single-query shapes that span several chunks, several rounds of the persistent kernel, ragged tails
    (4, 8, 8, 128, 2100, 1, [2049, 2100, 1, 127]),
    (2, 28, 4, 128, 1000, 1, [999, 513]),
    (40, 8, 8, 128, 704, 1, [704 - 13 * (i % 7) for i in range(40)]),
    (1, 8, 1, 128, 16400, 1, [16385]),
    (2, 6, 2, 128, 384, 1, [384, 256]),
    # blocks of queries on the tensor-core prefill path: several row blocks and key tiles, ragged tails,
    # a sequence shorter than two tiles, a group size that does not fill a row block
    (2, 16, 2, 128, 1200, 128, [1200, 777]),
    (1, 8, 1, 128, 700, 512, [699]),
    (2, 14, 2, 128, 300, 16, [16, 259]),
    (1, 24, 8, 128, 2200, 32, [2177]),
]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("mode", ["last_query", "chunk_sum", "accum", "external"])
@pytest.mark.parametrize("shape", SHAPES)
def test_score_matches_oracle(shape, mode, dtype):
    B, Hq, Hkv, d, cap, m, lens = shape
    seed = SHAPES.index(shape) * 10 + ["last_query", "chunk_sum", "accum", "external"].index(mode)
    q, K, V, lens_t = make_case(seed, B, Hq, Hkv, d, cap, m, dtype, lens)
    base = None
    if mode in ("accum", "external"):
        g = torch.Generator(device="cpu").manual_seed(5)
        base = (torch.rand((B, Hkv, cap), generator=g) * 4.0).to(DEV)
    base_in = None if base is None else base.clone()
    p, ws, o, scores = run_score(q, K, V, lens_t, m, mode, base)
    r = oracle_for(q, K, V, lens_t, scale=d ** -0.5, n_new=m, base_mode=mode, base=base_in)
    check_scores_and_o(r, scores, o, lens_t, f"{shape} {mode}")
    sc = f32(scores)
    for b, n in enumerate(lens):
        assert (sc[b, :, n:] == -7.0).all(), "slots behind the length must stay untouched"
        assert (sc[b, :, :n] >= 0).all()
        if n == 0:
            assert torch.isnan(o[b].float()).all(), "an empty sequence must be skipped"
    if mode == "accum":
        bg = f32(base)
        for b, n in enumerate(lens):
            assert_close(bg[b, :, :n], r["base"][b, :, :n], "accumulated base", rtol=1e-5, atol=1e-6)
            np.testing.assert_array_equal(bg[b, :, n:], f32(base_in)[b, :, n:])
    if mode == "external":
        assert torch.equal(base, base_in)
    # a second run is bit-identical (fixed reduction order, no atomics on floats)
    base2 = None if base_in is None else base_in.clone()
    _, _, o2, scores2 = run_score(q, K, V, lens_t, m, mode, base2)
    assert torch.equal(scores2, scores) and torch.equal(o2.view(torch.int32), o.view(torch.int32))


@pytest.mark.parametrize("mode", ["last_query", "accum"])
def test_decode_items_of_several_tiles_with_late_large_logits(mode):
    """Enough tiles that the decode kernel works in items of two tiles, with keys planted in the second
    tile of an item that top everything before them by far more than 2^8: the running softmax reference
    has to move and the output accumulated so far has to be rescaled. Sampled units against the oracle."""
    B, Hq, Hkv, d, cap = 10, 32, 8, 128, 1280
    G = Hq // Hkv
    lens = [1280 - 37 * (i % 5) for i in range(B)]
    q, K, V, lens_t = make_case(777, B, Hq, Hkv, d, cap, 1, torch.bfloat16, lens)
    units = [(0, 0), (3, 5), (9, 7), (6, 2)]
    for b, h in units:
        K[b, h, 200] = (q[b, h * G, 0].float() * 3.0).to(K.dtype)       # tile 1: ~ +49 in the log2 domain
        K[b, h, 450] = (q[b, h * G + 1, 0].float() * 1.0).to(K.dtype)   # tile 3: ~ +16
        K[b, h, 700] = (q[b, h * G + 3, 0].float() * 2.0).to(K.dtype)   # tile 5: ~ +33
    base = None
    if mode == "accum":
        g = torch.Generator(device="cpu").manual_seed(9)
        base = (torch.rand((B, Hkv, cap), generator=g) * 2.0).to(DEV)
    base_in = None if base is None else base.clone()
    p, ws, o, scores = run_score(q, K, V, lens_t, 1, mode, base)
    qs, Ks, Vs, ls, bs = sub_problem(q, K, V, lens_t, base_in, units, Hkv, G)
    r = oracle.score(f32(qs), f32(Ks), f32(Vs), ls.cpu().numpy(), scale=d ** -0.5, n_new=1, base_mode=mode,
                     base=None if bs is None else bs.double().cpu().numpy())
    sg, og = f32(scores), f32(o)
    for i, (b, h) in enumerate(units):
        n = lens[b]
        assert_close(sg[b, h, :n], r["scores"][i, 0, :n], f"unit ({b},{h}) scores")
        assert_close(og[b, h * G:(h + 1) * G], r["o"][i], f"unit ({b},{h}) o")


def test_c1_full_step_every_token():
    """Tiny fp32 configuration: scores of all 256 tokens, then evict 128 in one selection."""
    w = wl.WORKLOADS["c1"]
    K0, V0 = wl.initial_cache(w, DEV)
    q, kn, vn = wl.step_inputs(w, DEV, 0)
    cache = P.EvictionCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, 1, torch.float32,
                            w.budget, "last_query", "stable", max_evict=128)
    cache.load(K0, V0, wl.initial_lengths(w, DEV))
    P.caote_append(cache.params, cache.K, cache.V, cache.base, cache.pos, cache.lens, cache.n_seen, kn, vn,
                   cache.workspace)
    K1, V1, lens1 = cache.K.clone(), cache.V.clone(), cache.lens.clone()
    assert lens1.tolist() == [256]
    P.caote_score(cache.params, q, cache.K, cache.V, cache.lens, None, cache.o, cache.scores, cache.workspace)
    r = oracle_for(q, K1, V1, lens1, scale=w.scale, n_new=1, base_mode="last_query")
    assert_close(f32(cache.scores)[0, :, :256], r["scores"][0, :, :256], "c1 scores", rtol=2e-5, atol=1e-7)
    assert_close(f32(cache.o), r["o"], "c1 o", rtol=2e-5, atol=1e-6)
    P.caote_select_evict(cache.params, cache.scores, cache.lens, cache.budget, cache.pos, cache.evict_idx,
                         cache.n_evict, cache.workspace)
    assert cache.n_evict.tolist() == [128]
    pos = cache.pos.cpu().numpy()
    ev = cache.evict_idx.cpu().numpy()
    for h in range(w.n_kv_heads):
        check_evicted(r["scores"][0, h], pos[0, h], 256, 128, ev[0, h], f"c1 head {h}")
    P.caote_compact(cache.params, cache.K, cache.V, cache.base, cache.pos, cache.lens, cache.evict_idx,
                    cache.n_evict, "stable", cache.workspace)
    assert cache.lens.tolist() == [128] and cache.status() == 0
    for h in range(w.n_kv_heads):
        keep = np.setdiff1d(np.arange(256), ev[0, h])
        assert torch.equal(cache.K[0, h, :128].cpu(), K1[0, h].cpu()[keep])
        assert torch.equal(cache.V[0, h, :128].cpu(), V1[0, h].cpu()[keep])
        assert cache.pos[0, h, :128].cpu().tolist() == keep.tolist()


@pytest.mark.parametrize("n,k", [(1, 0), (5, 0), (5, 1), (5, 4), (1000, 1), (1000, 37), (1000, 999),
                                 (4224, 128), (16896, 512), (3000, 1500)])
@pytest.mark.parametrize("ties", [False, True])
def test_select_is_bit_exact(n, k, ties):
    B, Hkv, cap = 2, 3, n + 3
    g = torch.Generator(device="cpu").manual_seed(n * 7 + k)
    scores = torch.rand((B, Hkv, cap), generator=g)
    if ties:
        scores = (scores * 8).floor() / 8
        scores[0, 0, : n // 2] = 0.0
        scores[1, 1, :] = float("inf")
    pos = torch.stack([torch.stack([torch.randperm(cap, generator=g) for _ in range(Hkv)]) for _ in range(B)])
    lens = torch.tensor([n, max(n - 1, 1)], dtype=torch.int32)
    budget = torch.tensor([n - k, max(n - 1, 1) - min(k, max(n - 2, 0))], dtype=torch.int32).clamp(min=1)
    p = P.make_params(B, Hkv, Hkv, 64, cap, 1, torch.float32, 1.0, "last_query")
    ws = P.alloc_workspace(p, DEV)
    max_evict = max(k, 1)
    for use_pos in (True, False):
        ev = torch.full((B, Hkv, max_evict), -1, dtype=torch.int32, device=DEV)
        ne = torch.full((B,), -1, dtype=torch.int32, device=DEV)
        pos_d = pos.to(torch.int32).to(DEV) if use_pos else None
        P.caote_select_evict(p, scores.to(DEV), lens.to(DEV), budget.to(DEV), pos_d, ev, ne, ws)
        assert P.caote_read_status(ws) == 0
        ref, kref = oracle.select_evict(scores.numpy(), lens.numpy(), budget.numpy(),
                                        pos.numpy() if use_pos else None)
        assert ne.cpu().tolist() == kref.tolist()
        evc = ev.cpu().numpy()
        for b in range(B):
            for h in range(Hkv):
                assert evc[b, h, :kref[b]].tolist() == ref[b][h].tolist()
                assert (evc[b, h, kref[b]:] == -1).all()


@pytest.mark.parametrize("mode", ["fill", "stable"])
@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 64)])
@pytest.mark.parametrize("n,k", [(10, 0), (10, 1), (10, 9), (777, 128), (777, 1), (300, 299), (2000, 700)])
def test_compact_preserves_the_survivors(mode, dtype, d, n, k):
    B, Hkv, cap = 2, 2, n + 5
    g = torch.Generator(device="cpu").manual_seed(n + k)
    K = torch.randn((B, Hkv, cap, d), generator=g).to(dtype).to(DEV)
    V = torch.randn((B, Hkv, cap, d), generator=g).to(dtype).to(DEV)
    base = torch.rand((B, Hkv, cap), generator=g).to(DEV)
    pos = torch.arange(cap, dtype=torch.int32).expand(B, Hkv, cap).contiguous().to(DEV) + 100
    lens = torch.tensor([n, n - 1 if n > k + 1 else n], dtype=torch.int32, device=DEV)
    K0, V0, base0, pos0, lens0 = K.clone(), V.clone(), base.clone(), pos.clone(), lens.clone()
    ne = torch.tensor([k, k], dtype=torch.int32, device=DEV)
    ev = torch.zeros((B, Hkv, max(k, 1)), dtype=torch.int32)
    for b in range(B):
        for h in range(Hkv):
            nb = int(lens0[b])
            ev[b, h, :k] = torch.sort(torch.randperm(nb, generator=g)[:k]).values
    p = P.make_params(B, Hkv, Hkv, d, cap, 1, dtype, 1.0, "last_query")
    ws = P.alloc_workspace(p, DEV)
    P.caote_compact(p, K, V, base, pos, lens, ev.to(DEV), ne, mode, ws)
    assert P.caote_read_status(ws) == 0
    assert lens.cpu().tolist() == (lens0.cpu() - k).tolist()
    for b in range(B):
        for h in range(Hkv):
            nb, nn = int(lens0[b]), int(lens0[b]) - k
            keep = np.setdiff1d(np.arange(nb), ev[b, h, :k].numpy())
            got_pos = pos[b, h, :nn].cpu().numpy()
            if mode == "stable":
                assert got_pos.tolist() == (keep + 100).tolist()
            else:
                assert sorted(got_pos.tolist()) == (keep + 100).tolist()
            src = torch.from_numpy(got_pos - 100).long()
            assert torch.equal(K[b, h, :nn].cpu(), K0[b, h].cpu()[src])
            assert torch.equal(V[b, h, :nn].cpu(), V0[b, h].cpu()[src])
            assert torch.equal(base[b, h, :nn].cpu(), base0[b, h].cpu()[src])


def test_append_and_status_word():
    B, Hq, Hkv, d, cap, m = 2, 4, 2, 64, 20, 3
    p = P.make_params(B, Hq, Hkv, d, cap, m, torch.bfloat16, 0.125, "accum")
    ws = P.alloc_workspace(p, DEV)
    K = torch.zeros((B, Hkv, cap, d), dtype=torch.bfloat16, device=DEV)
    V = torch.zeros_like(K)
    base = torch.ones((B, Hkv, cap), device=DEV)
    pos = torch.full((B, Hkv, cap), -1, dtype=torch.int32, device=DEV)
    lens = torch.tensor([4, 18], dtype=torch.int32, device=DEV)  # 18 + 3 > 20 -> skipped
    seen = torch.tensor([40, 50], dtype=torch.int32, device=DEV)
    kn = torch.randn((B, Hkv, m, d), device=DEV).to(torch.bfloat16)
    vn = torch.randn((B, Hkv, m, d), device=DEV).to(torch.bfloat16)
    P.caote_append(p, K, V, base, pos, lens, seen, kn, vn, ws)
    assert P.caote_read_status(ws) == P.binding.ERR_OVERFLOW
    assert P.caote_read_status(ws) == 0  # reading resets it
    assert lens.tolist() == [7, 18] and seen.tolist() == [43, 50]
    assert torch.equal(K[0, :, 4:7], kn[0]) and torch.equal(V[0, :, 4:7], vn[0])
    assert (K[1] == 0).all() and (base[0, :, 4:7] == 0).all() and (base[1] == 1).all()
    assert pos[0, 0, 4:7].tolist() == [40, 41, 42]
    # a length beyond capacity or below n_new is reported, not dereferenced
    q = torch.randn((B, Hq, m, d), device=DEV).to(torch.bfloat16)
    o = torch.zeros(q.shape, device=DEV)
    scores = torch.zeros((B, Hkv, cap), device=DEV)
    bad = torch.tensor([2, 21], dtype=torch.int32, device=DEV)
    P.caote_score(p, q, K, V, bad, base, o, scores, ws)
    assert P.caote_read_status(ws) == P.binding.ERR_BAD_LENGTH
    # more evictions than max_evict
    ev = torch.zeros((B, Hkv, 2), dtype=torch.int32, device=DEV)
    ne = torch.zeros((B,), dtype=torch.int32, device=DEV)
    P.caote_select_evict(p, scores, lens, torch.tensor([1, 17], dtype=torch.int32, device=DEV), None, ev, ne, ws)
    assert P.caote_read_status(ws) == P.binding.ERR_OVERFLOW
    assert ne.tolist() == [0, 1]


def dominant_case(seed, B, Hq, Hkv, d, cap, m, dtype, lens, eps, slot):
    """Every query row of every head is (nearly) the same vector q0 and one key per unit is c * q0, with c chosen
    so that this key takes all but about `eps` of every row's weight: 1 - w_j ~ eps must then not be formed by
    cancellation."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    q0 = torch.randn((B, Hkv, 1, 1, d), generator=g)
    q = (q0 + 0.02 * torch.randn((B, Hkv, Hq // Hkv, m, d), generator=g)).reshape(B, Hq, m, d)
    K = torch.randn((B, Hkv, cap, d), generator=g)
    V = torch.randn((B, Hkv, cap, d), generator=g)
    for b in range(B):
        for h in range(Hkv):
            v0 = q0[b, h, 0, 0]
            others = torch.exp((K[b, h, :lens[b]] @ v0) * d ** -0.5).sum()  # the other keys' numerators for q0
            logit = float(torch.log(others / eps))
            K[b, h, slot] = v0 * (logit / (d ** -0.5 * float(v0 @ v0)))
    return (q.to(dtype).to(DEV), K.to(dtype).to(DEV), V.to(dtype).to(DEV),
            torch.tensor(lens, dtype=torch.int32, device=DEV))


@pytest.mark.parametrize("eps", [1e-1, 1e-2, 1e-3, 1e-4])
@pytest.mark.parametrize("shape", [
    # B, Hq, Hkv, d, cap, m, lens, mode, dtype            path
    (2, 8, 2, 128, 1600, 1, [1531, 700], "last_query", torch.bfloat16),   # single query, G 4
    (1, 7, 1, 128, 9000, 1, [8193], "accum", torch.bfloat16),             # single query, G 7, carried base scores
    (2, 8, 1, 128, 300, 1, [257, 300], "last_query", torch.bfloat16),     # single query, G 8, few tiles
    (1, 8, 2, 128, 700, 128, [640], "chunk_sum", torch.bfloat16),         # block of queries, tensor-core path
    (1, 4, 2, 64, 200, 3, [150], "chunk_sum", torch.float32),             # any-shape path
    (1, 4, 2, 64, 200, 1, [190], "last_query", torch.float32),            # any-shape path, one query
])
def test_token_holding_almost_all_the_weight(shape, eps):
    """One token of every unit holds all but ~eps of the weight (Sec. 3.2 normalisation; the oracle forms 1 - w_j
    as the sum of the other weights). Down to eps = 1e-3 its score and everybody else's stay within the stated
    tolerance. At 1e-4 the planted token's own score is bounded by something else: X - v_j is then a difference
    of two fp32 vectors that agree to four digits, which leaves the distance about three digits; it is held
    to 2e-2 there, everybody else to the stated tolerance."""
    B, Hq, Hkv, d, cap, m, lens, mode, dtype = shape
    slot = 77
    q, K, V, lens_t = dominant_case(int(-np.log10(eps)) * 31 + Hq, B, Hq, Hkv, d, cap, m, dtype, lens, eps, slot)
    base = None
    if mode == "accum":
        g = torch.Generator(device="cpu").manual_seed(3)
        base = (torch.rand((B, Hkv, cap), generator=g) * 1e-9).to(DEV)
    base_in = None if base is None else base.clone()
    p, ws, o, scores = run_score(q, K, V, lens_t, m, mode, base)
    r = oracle_for(q, K, V, lens_t, scale=d ** -0.5, n_new=m, base_mode=mode, base=base_in)
    for b in range(B):
        comp = 1.0 - r["w"][b, :, slot]
        assert (comp < 6 * eps).all() and (comp > eps / 6).all(), f"construction: 1 - w = {comp}, wanted ~{eps}"
    if eps >= 1e-3:
        check_scores_and_o(r, scores, o, lens_t, f"{shape} eps {eps}")
    else:
        sg = f32(scores).astype(np.float64)
        for b, n in enumerate(lens):
            rest = np.ones(n, dtype=bool)
            rest[slot] = False
            assert_close(sg[b, :, :n][:, rest], r["scores"][b, :, :n][:, rest], f"{shape} eps {eps} others")
            assert_close(sg[b, :, slot], r["scores"][b, :, slot], f"{shape} eps {eps} planted token", rtol=2e-2)
            assert_close(f32(o)[b], r["o"][b], "o")


@pytest.mark.parametrize("mode,m,dtype,d", [("last_query", 1, torch.bfloat16, 128), ("accum", 1, torch.bfloat16, 128),
                                            ("chunk_sum", 64, torch.bfloat16, 128), ("chunk_sum", 2, torch.float32, 64)])
def test_equal_values_and_dominant_base_score(mode, m, dtype, d):
    """All value rows equal: X equals every v_j up to the rounding of the accumulated output, so every score is
    (within the absolute tolerance) zero. And a carried base score that holds almost all of the normaliser
    (accumulated mode, single-query path) keeps an accurate complement."""
    B, Hq, Hkv, cap, n = 1, 8, 2, 1500, 1409
    q, K, V, lens_t = make_case(91, B, Hq, Hkv, d, cap, m, dtype, [n])
    Veq = V[:, :, :1].expand_as(V).contiguous()
    gen0 = torch.Generator(device=DEV)
    gen0.manual_seed(90)
    base = torch.rand((B, Hkv, cap), device=DEV, generator=gen0) if mode == "accum" else None
    base_in = None if base is None else base.clone()
    _, _, o, scores = run_score(q, K, Veq, lens_t, m, mode, base)
    r = oracle_for(q, K, Veq, lens_t, scale=d ** -0.5, n_new=m, base_mode=mode, base=base_in)
    assert np.abs(r["scores"][0, :, :n]).max() < 1e-12
    check_scores_and_o(r, scores, o, lens_t, "equal values")
    if mode == "accum":
        # 1 - w of the planted token is about 4e-4: above the 1e-4 below which fp32 itself (the rounding of X next
        # to v_j, about 1e-7 / (1 - w) relative) decides the result on every path
        gen = torch.Generator(device=DEV)
        gen.manual_seed(92)
        base = torch.rand((B, Hkv, cap), device=DEV, generator=gen) * 1e-2
        base[:, :, 500] = 3e4
        base_in = base.clone()
        _, _, o, scores = run_score(q, K, V, lens_t, m, mode, base)
        r = oracle_for(q, K, V, lens_t, scale=d ** -0.5, n_new=m, base_mode=mode, base=base_in)
        assert (1.0 - r["w"][0, :, 500] < 1e-3).all()
        check_scores_and_o(r, scores, o, lens_t, "dominant carried base score")


def test_a_wait_that_runs_out_is_reported_and_the_library_stays_usable():
    """The single-query kernel bounds every device-side wait by a clock limit. With the limit set far below the
    latency of a memory copy the waits for the first tiles run out: the call must still return, record
    CAOTE_ERR_TIMEOUT in the status word, and leave the library, the workspace and the caches usable - the same
    call with the default limit then gives the oracle's result."""
    B, Hq, Hkv, d, cap = 6, 8, 2, 128, 1100
    lens = [1031, 900, 1100, 513, 1024, 257]
    q, K, V, lens_t = make_case(4242, B, Hq, Hkv, d, cap, 1, torch.bfloat16, lens)
    p = P.make_params(B, Hq, Hkv, d, cap, 1, torch.bfloat16, d ** -0.5, "last_query")
    ws = P.alloc_workspace(p, DEV)
    o = torch.zeros(q.shape, dtype=torch.float32, device=DEV)
    scores = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=DEV)
    P.caote_set_option(P.binding.OPT_WAIT_CYCLES, 200)
    try:
        P.caote_score(p, q, K, V, lens_t, None, o, scores, ws)
        torch.cuda.synchronize()  # the call came back
        assert P.caote_read_status(ws) == P.binding.ERR_TIMEOUT
    finally:
        P.caote_set_option(P.binding.OPT_WAIT_CYCLES, 2_000_000_000)
    assert P.caote_read_status(ws) == 0  # reading resets the word
    P.caote_score(p, q, K, V, lens_t, None, o, scores, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    r = oracle_for(q, K, V, lens_t, scale=d ** -0.5, n_new=1, base_mode="last_query")
    check_scores_and_o(r, scores, o, lens_t, "after a timed-out call")
