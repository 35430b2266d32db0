"""The five benchmark configurations, stepped on the GPU through the C ABI and checked in lock-step.

Before every step the cache state the GPU is about to work on is copied out; the oracle then scores
exactly that state plus the step's new tokens, so one tolerated near-threshold difference in an evicted
set cannot cascade into later steps. Scores and attention outputs are compared element by element,
evicted sets with the band rule of tests/parity.py, and the compacted cache through `pos`.

Configurations 3-5 are run at reduced size for the element-by-element trajectory (the oracle is a plain
triple loop) and once at full size, in the launch configuration the benchmark times, with the oracle
following a seeded sample of (sequence, KV head) units - units are independent.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_14051_b200 as P
from paper_2504_14051_b200 import workloads as wl

from parity import assert_close, check_evicted, f32, sub_problem

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_cache(w, compact="fill"):
    lens0 = wl.initial_lengths(w, DEV)
    budget = lens0.clone() if w.ragged_min_len is not None else torch.full_like(lens0, w.budget)
    c = P.EvictionCache(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.capacity, w.n_new, w.torch_dtype, budget,
                        w.base_mode, compact, w.scale, max_evict=w.n_new, device=DEV)
    K0, V0 = wl.initial_cache(w, DEV)
    c.load(K0, V0, lens0)
    return c


def lockstep(w, steps, units=None, compact="fill", random_base=False):
    """Run `steps` steps; check every step against the oracle on `units` (default: all). random_base: the carried
    base scores start from seeded positive values instead of zero (a cache that has been running for a while)."""
    c = make_cache(w, compact)
    if random_base:
        g = torch.Generator(device="cpu").manual_seed(w.seed + 1)
        c.base.copy_((torch.rand(c.base.shape, generator=g) * 3.0).to(DEV))
    G, Hkv, m = w.group, w.n_kv_heads, w.n_new
    if units is None:
        units = [(b, h) for b in range(w.batch) for h in range(Hkv)]
    flips = 0
    for t in range(steps):
        q, kn, vn = wl.step_inputs(w, DEV, t)
        # the state the step starts from, with the new tokens appended the way caote_step will
        K, V, lens = c.K.clone(), c.V.clone(), c.lens.clone()
        base, pos = c.base.clone(), c.pos.clone()
        seen = c.n_seen.clone()
        for b in range(w.batch):
            n = int(lens[b])
            K[b, :, n:n + m], V[b, :, n:n + m] = kn[b], vn[b]
            base[b, :, n:n + m] = 0.0
            pos[b, :, n:n + m] = (seen[b] + torch.arange(m, device=DEV, dtype=torch.int32))[None, :]
        lens = lens + m
        o = c.step(q, kn, vn).clone()
        assert c.status() == 0
        qs, Ks, Vs, ls, bs = sub_problem(q, K, V, lens, base if w.base_mode in ("accum", "external") else None,
                                         units, Hkv, G)
        r = oracle.score(f32(qs), f32(Ks), f32(Vs), ls.cpu().numpy(), scale=w.scale, n_new=m, base_mode=w.base_mode,
                         base=None if bs is None else bs.double().cpu().numpy())
        sc, ev, ne = f32(c.scores), c.evict_idx.cpu().numpy(), c.n_evict.cpu().numpy()
        og, posn, lens_after = f32(o), pos.cpu().numpy(), c.lens.cpu().numpy()
        budget = c.budget.cpu().numpy()
        for i, (b, h) in enumerate(units):
            n = int(lens[b])
            what = f"{w.name} step {t} unit ({b},{h})"
            assert_close(sc[b, h, :n], r["scores"][i, 0, :n], what + " scores")
            assert_close(og[b, h * G:(h + 1) * G], r["o"][i], what + " o")
            k = max(0, n - int(budget[b]))
            assert int(ne[b]) == k and int(lens_after[b]) == n - k
            flips += check_evicted(r["scores"][i, 0], posn[b, h], n, k, ev[b, h, :k], what)
            # the compacted cache holds exactly the survivors
            keep = np.setdiff1d(np.arange(n), ev[b, h, :k])
            got = np.sort(c.pos[b, h, :n - k].cpu().numpy())
            np.testing.assert_array_equal(got, np.sort(posn[b, h, keep]))
            # ... and their K and V rows moved with them: slot i of the compacted cache holds the row of the slot that
            # had its position before the step
            by_pos = np.argsort(posn[b, h, :n])
            src = by_pos[np.searchsorted(posn[b, h, :n][by_pos], c.pos[b, h, :n - k].cpu().numpy())]
            src_t = torch.as_tensor(src, device=DEV)
            assert torch.equal(c.K[b, h, :n - k], K[b, h][src_t]), what + " K rows after compaction"
            assert torch.equal(c.V[b, h, :n - k], V[b, h][src_t]), what + " V rows after compaction"
            if compact == "stable":
                assert (np.diff(src) > 0).all(), what + " order of the survivors"
            if w.base_mode == "accum":
                order = np.argsort(c.pos[b, h, :n - k].cpu().numpy())
                ref_b = r["base"][i, 0, keep][np.argsort(posn[b, h, keep])]
                assert_close(f32(c.base)[b, h, :n - k][order], ref_b, what + " carried base", rtol=1e-4, atol=1e-6)
    return flips


def test_c2_decode_with_sinks_lockstep():
    w = wl.scaled(wl.WORKLOADS["c2"], steps=64)
    lockstep(w, 64)


def test_c3_chunked_prefill_reduced_lockstep():
    w = wl.scaled(wl.WORKLOADS["c3"], budget=1024, init_len=1024, layers=1)
    lockstep(w, 6)


def test_c3_chunked_prefill_fills_before_it_evicts():
    w = wl.scaled(wl.WORKLOADS["c3"], budget=384, init_len=0, layers=1)
    lockstep(w, 4, units=[(0, 0), (0, 5)])  # 128, 256, 384 tokens: no eviction; then 512 -> evict 128


def test_c4_ragged_accumulated_reduced_lockstep():
    w = wl.scaled(wl.WORKLOADS["c4"], batch=3, budget=1500, init_len=1500, ragged_min_len=1100)
    lockstep(w, 32)


def test_c5_prefill_then_decode_reduced_lockstep():
    wp = wl.scaled(wl.WORKLOADS["c5p"], batch=1, budget=1536, init_len=1536)
    lockstep(wp, 1, units=[(0, 0), (0, 7)])
    wd = wl.scaled(wl.WORKLOADS["c5d"], batch=2, budget=1536, init_len=1536)
    lockstep(wd, 16)


@pytest.mark.parametrize("name,units", [
    ("c4", [(0, 0), (17, 3), (63, 1)]),
    ("c5d", [(0, 0), (7, 7)]),
    ("c3", [(0, 2)]),
    ("c5p", [(3, 5)]),
])
def test_full_size_step_on_sampled_units(name, units):
    """One step at the size and launch configuration the benchmark times; the oracle follows a sample."""
    w = wl.WORKLOADS[name]
    if w.n_new > 1:
        w = wl.scaled(w, init_len=w.budget, layers=1)
    lockstep(w, 1, units=units)


def test_full_size_c4_steps_with_carried_base_scores():
    """Two full-size steps of the accumulated-score workload starting from non-zero carried base scores (row 7 of
    the P operand and the base tiles staged beside the value tiles are in play from the first launch on)."""
    lockstep(wl.WORKLOADS["c4"], 2, units=[(5, 2), (40, 0), (63, 3)], random_base=True)
