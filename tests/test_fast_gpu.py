"""FastCAOTE (Sec. 3.3) on the GPU against the oracle: scores with X = mean of the cached values, and the
running per-unit sum of value rows that the library carries from step to step."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_14051_b200 as P
from paper_2504_14051_b200 import workloads as wl

from parity import assert_close, check_evicted, f32, sub_problem
from test_gpu_parity import make_case

pytestmark = pytest.mark.gpu
DEV = "cuda"

SHAPES = [
    # B, Hq, Hkv, d, cap, m, lens, dtype      (path)
    (2, 8, 2, 128, 300, 1, [257, 129], torch.bfloat16),        # single-query tensor-core path
    (1, 7, 1, 128, 1100, 1, [1031], torch.bfloat16),
    (3, 16, 2, 128, 200, 1, [200, 0, 65], torch.bfloat16),
    (10, 32, 8, 128, 1280, 1, [1280 - 37 * (i % 5) for i in range(10)], torch.bfloat16),  # items of two tiles
    (2, 16, 2, 128, 1200, 128, [1200, 777], torch.bfloat16),   # tensor-core prefill path
    (2, 4, 2, 64, 80, 1, [63, 80], torch.float32),             # generic path
    (1, 14, 2, 128, 400, 3, [333], torch.bfloat16),
]


def expected_fast(r, V, lens, units):
    out = {}
    Vf = f32(V)
    for b, h in units:
        n = int(lens[b])
        out[(b, h)] = oracle.fast_scores(r["w"][b, h, :n], Vf[b, h, :n]) if n > 0 else np.zeros(0)
    return out


@pytest.fixture(params=["cluster", "streaming"])
def single_query_kernel(request):
    """Single-query shapes take the cluster kernel by default; with it switched off they take the streaming
    variant, which otherwise only units beyond the cluster kernel's reach would."""
    if request.param == "streaming":
        P.caote_set_option(P.OPT_DECODE_CLUSTER, -1)
    yield request.param
    P.caote_set_option(P.OPT_DECODE_CLUSTER, 0)


@pytest.mark.parametrize("mode", ["last_query", "chunk_sum", "accum", "external"])
@pytest.mark.parametrize("shape", SHAPES)
def test_fast_scores_match_oracle(shape, mode, single_query_kernel):
    B, Hq, Hkv, d, cap, m, lens, dtype = shape
    if single_query_kernel == "streaming" and (m != 1 or dtype != torch.bfloat16):
        pytest.skip("the option only changes single-query bf16 shapes")
    q, K, V, lens_t = make_case(4242 + SHAPES.index(shape), B, Hq, Hkv, d, cap, m, dtype, lens)
    base = None
    if mode in ("accum", "external"):
        g = torch.Generator(device="cpu").manual_seed(5)
        base = (torch.rand((B, Hkv, cap), generator=g) * 4.0).to(DEV)
    base_in = None if base is None else base.clone()
    p = P.make_params(B, Hq, Hkv, d, cap, m, dtype, d ** -0.5, mode)
    ws = P.alloc_workspace(p, DEV)
    vsum = torch.full((B, Hkv, d), float("nan"), dtype=torch.float32, device=DEV)
    P.caote_vsum(p, V, lens_t, vsum)
    for b, n in enumerate(lens):
        ref = V[b, :, :n].double().sum(dim=1)
        assert_close(vsum[b].double().cpu().numpy(), ref.cpu().numpy(), "vsum", rtol=1e-5, atol=1e-3)
    o = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    scores = torch.full((B, Hkv, cap), -7.0, dtype=torch.float32, device=DEV)
    P.caote_score_fast(p, q, K, V, lens_t, base, vsum, o, scores, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    r = oracle.score(f32(q), f32(K), f32(V), lens_t.cpu().numpy(), scale=d ** -0.5, n_new=m, base_mode=mode,
                     base=None if base_in is None else base_in.double().cpu().numpy())
    units = [(b, h) for b in range(B) for h in range(Hkv)]
    exp = expected_fast(r, V, lens, units)
    sg, og = f32(scores), f32(o)
    for b, h in units:
        n = lens[b]
        if n == 0:
            continue
        assert_close(sg[b, h, :n], exp[(b, h)], f"{shape} {mode} fast scores ({b},{h})")
        assert (sg[b, h, n:] == -7.0).all()
    for b, n in enumerate(lens):
        if n:
            assert_close(og[b], r["o"][b], f"{shape} {mode} o[b={b}]")
    if mode == "accum":
        for b, n in enumerate(lens):
            assert_close(f32(base)[b, :, :n], r["base"][b, :, :n], "accumulated base", rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("name,kw,steps,compact", [
    ("c4", dict(batch=3, budget=1500, init_len=1500, ragged_min_len=1100), 4, "fill"),
    ("c4", dict(batch=2, budget=700, init_len=700, ragged_min_len=600), 3, "stable"),
    ("c3", dict(budget=1024, init_len=1024, layers=1), 2, "fill"),
])
def test_fast_steps_keep_the_sum_current(name, kw, steps, compact):
    """Several steps through caote_step_fast: before each step the state is copied out and the oracle scores
    it; the running sum must equal the sum of the valid V rows after every step."""
    w = wl.scaled(wl.WORKLOADS[name], **kw)
    G, Hkv, m = w.group, w.n_kv_heads, w.n_new
    lens0 = wl.initial_lengths(w, DEV)
    budget = lens0.clone() if w.ragged_min_len is not None else torch.full_like(lens0, w.budget)
    c = P.EvictionCache(w.batch, w.n_q_heads, Hkv, w.head_dim, w.capacity, m, w.torch_dtype, budget, w.base_mode, compact,
                        w.scale, max_evict=m, device=DEV, method="fast")
    K0, V0 = wl.initial_cache(w, DEV)
    c.load(K0, V0, lens0)
    units = [(b, h) for b in range(w.batch) for h in range(Hkv)][:6]
    for t in range(steps):
        q, kn, vn = wl.step_inputs(w, DEV, t)
        K, V, lens = c.K.clone(), c.V.clone(), c.lens.clone()
        base, pos, seen = c.base.clone(), c.pos.clone(), c.n_seen.clone()
        for b in range(w.batch):
            n = int(lens[b])
            K[b, :, n:n + m], V[b, :, n:n + m] = kn[b], vn[b]
            base[b, :, n:n + m] = 0.0
            pos[b, :, n:n + m] = (seen[b] + torch.arange(m, device=DEV, dtype=torch.int32))[None, :]
        lens = lens + m
        c.step(q, kn, vn)
        assert c.status() == 0
        qs, Ks, Vs, ls, bs = sub_problem(q, K, V, lens, base if w.base_mode in ("accum", "external") else None, units, Hkv, G)
        r = oracle.score(f32(qs), f32(Ks), f32(Vs), ls.cpu().numpy(), scale=w.scale, n_new=m, base_mode=w.base_mode,
                         base=None if bs is None else bs.double().cpu().numpy())
        sc, ev, posn = f32(c.scores), c.evict_idx.cpu().numpy(), pos.cpu().numpy()
        for i, (b, h) in enumerate(units):
            n = int(lens[b])
            ref = oracle.fast_scores(r["w"][i, 0, :n], f32(Vs)[i, 0, :n])
            assert_close(sc[b, h, :n], ref, f"{name} step {t} unit ({b},{h}) fast scores")
            k = max(0, n - int(c.budget[b]))
            check_evicted(ref, posn[b, h], n, k, ev[b, h, :k], f"{name} step {t} unit ({b},{h})")
        for b in range(w.batch):
            n = int(c.lens[b])
            ref = c.V[b, :, :n].double().sum(dim=1).cpu().numpy()
            assert_close(c.vsum[b].double().cpu().numpy(), ref, f"{name} step {t} vsum[b={b}]", rtol=1e-5, atol=2e-3)


def test_fast_scores_rank_like_caote_scores():
    """Sec. 3.3 reports a Spearman correlation >= 0.8 between FastCAOTE and CAOTE scores on real models.
    Here: the same check on synthetic decode caches (keys partly aligned with the queries, so that the
    weights are far from uniform), on the GPU's scores, with the oracle's correlation beside it."""
    from scipy.stats import spearmanr

    B, Hq, Hkv, d, cap = 4, 16, 4, 128, 1536
    lens = [1536, 1400, 1290, 1025]
    q, K, V, lens_t = make_case(99, B, Hq, Hkv, d, cap, 1, torch.bfloat16, lens)
    G = Hq // Hkv
    for b in range(B):            # every 16th key leans towards one of the unit's queries
        for h in range(Hkv):
            K[b, h, ::16] = (K[b, h, ::16].float() + 0.6 * q[b, h * G, 0].float()).to(K.dtype)
    p = P.make_params(B, Hq, Hkv, d, cap, 1, torch.bfloat16, d ** -0.5, "last_query")
    ws = P.alloc_workspace(p, DEV)
    o = torch.zeros(q.shape, dtype=torch.float32, device=DEV)
    caote = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=DEV)
    fast = torch.zeros_like(caote)
    vsum = torch.zeros((B, Hkv, d), dtype=torch.float32, device=DEV)
    P.caote_score(p, q, K, V, lens_t, None, o, caote, ws)
    P.caote_vsum(p, V, lens_t, vsum)
    P.caote_score_fast(p, q, K, V, lens_t, None, vsum, o, fast, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    r = oracle.score(f32(q), f32(K), f32(V), lens_t.cpu().numpy(), scale=d ** -0.5, n_new=1, base_mode="last_query")
    cg, fg, Vf = f32(caote), f32(fast), f32(V)
    for b in range(B):
        n = lens[b]
        for h in range(Hkv):
            rho_gpu = spearmanr(cg[b, h, :n], fg[b, h, :n]).statistic
            rho_ref = spearmanr(r["scores"][b, h, :n], oracle.fast_scores(r["w"][b, h, :n], Vf[b, h, :n])).statistic
            assert rho_gpu >= 0.8, f"unit ({b},{h}): Spearman {rho_gpu}"
            assert abs(rho_gpu - rho_ref) < 5e-3, f"unit ({b},{h}): GPU {rho_gpu} vs oracle {rho_ref}"


@pytest.mark.parametrize("name,units", [("c4", [(0, 0), (17, 3), (63, 1)]), ("c5d", [(7, 7)])])
def test_fast_full_size_step_on_sampled_units(name, units):
    """One FastCAOTE step at the size and launch configuration the benchmark times; the oracle follows a sample."""
    w = wl.WORKLOADS[name]
    G, Hkv, m = w.group, w.n_kv_heads, w.n_new
    lens0 = wl.initial_lengths(w, DEV)
    budget = lens0.clone() if w.ragged_min_len is not None else torch.full_like(lens0, w.budget)
    c = P.EvictionCache(w.batch, w.n_q_heads, Hkv, w.head_dim, w.capacity, m, w.torch_dtype, budget, w.base_mode, "fill",
                        w.scale, max_evict=m, device=DEV, method="fast")
    K0, V0 = wl.initial_cache(w, DEV)
    c.load(K0, V0, lens0)
    del K0, V0
    q, kn, vn = wl.step_inputs(w, DEV, 0)
    lens = c.lens.clone() + m
    sub = {}
    for b, h in units:  # the unit's state with the new token appended the way the step will
        n = int(lens[b])
        Ku, Vu = c.K[b, h, :n].clone(), c.V[b, h, :n].clone()
        Ku[n - m:], Vu[n - m:] = kn[b, h], vn[b, h]
        sub[(b, h)] = (Ku, Vu, c.base[b, h, :n].clone(), c.pos[b, h, :n].clone(), int(c.n_seen[b]))
    c.step(q, kn, vn)
    assert c.status() == 0
    sc, ev = f32(c.scores), c.evict_idx.cpu().numpy()
    for b, h in units:
        Ku, Vu, bu, pu, seen = sub[(b, h)]
        n = Ku.shape[0]
        bu[n - m:] = 0.0
        pu[n - m:] = seen + torch.arange(m, device=DEV, dtype=torch.int32)
        r = oracle.score(f32(q[b:b + 1, h * G:(h + 1) * G]), f32(Ku)[None, None], f32(Vu)[None, None], np.array([n], dtype=np.int32),
                         scale=w.scale, n_new=m, base_mode=w.base_mode,
                         base=bu.double().cpu().numpy()[None, None] if w.base_mode in ("accum", "external") else None)
        ref = oracle.fast_scores(r["w"][0, 0, :n], f32(Vu))
        assert_close(sc[b, h, :n], ref, f"{name} unit ({b},{h}) fast scores")
        assert_close(f32(c.o)[b, h * G:(h + 1) * G], r["o"][0], f"{name} unit ({b},{h}) o")
        k = max(0, n - int(c.budget[b]))
        check_evicted(ref, pu.cpu().numpy(), n, k, ev[b, h, :k], f"{name} unit ({b},{h})")


def test_a_sequence_without_room_keeps_its_running_sum():
    """caote_step_fast on single-query shapes adds the new value row to the running sum inside the append: a sequence
    whose cache has no room for the new token is skipped by the append (status: overflow), and its sum, its rows and
    its length stay as they were; the other sequence's sum takes its new row and gives up the evicted one."""
    B, Hq, Hkv, d, cap = 2, 8, 2, 128, 300
    g = torch.Generator(device="cpu").manual_seed(99)
    c = P.EvictionCache(B, Hq, Hkv, d, cap, 1, torch.bfloat16, torch.tensor([256, 300], dtype=torch.int32, device=DEV),
                        "last_query", "fill", d ** -0.5, max_evict=1, device=DEV, method="fast")
    K0 = torch.randn((B, Hkv, cap, d), generator=g).to(torch.bfloat16).to(DEV)
    V0 = torch.randn((B, Hkv, cap, d), generator=g).to(torch.bfloat16).to(DEV)
    c.load(K0, V0, torch.tensor([256, 300], dtype=torch.int32, device=DEV))  # the second one is full
    q = torch.randn((B, Hq, 1, d), generator=g).to(torch.bfloat16).to(DEV)
    kn = torch.randn((B, Hkv, 1, d), generator=g).to(torch.bfloat16).to(DEV)
    vn = torch.randn((B, Hkv, 1, d), generator=g).to(torch.bfloat16).to(DEV)
    vsum0, V1 = c.vsum.clone(), c.V.clone()
    c.step(q, kn, vn)
    torch.cuda.synchronize()
    assert c.status() == P.binding.ERR_OVERFLOW
    assert c.lens.tolist() == [256, 300] and c.n_evict.tolist() == [1, 0]
    assert torch.equal(c.vsum[1], vsum0[1]) and torch.equal(c.V[1], V1[1])
    ref = c.V[0, :, :256].double().sum(dim=1).cpu().numpy()
    assert_close(c.vsum[0].double().cpu().numpy(), ref, "running sum of the sequence that took its new row", rtol=1e-5, atol=2e-3)
