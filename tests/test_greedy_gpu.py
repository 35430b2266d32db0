"""GPU parity of greedy multi-token eviction (Appendix B chained) against the oracle's sequence.

The GPU's picks are followed in lock-step: as long as they agree with the oracle's greedy sequence nothing else
is needed; where they differ, the oracle scores the state the GPU was in (the tokens still present, weights
renormalised) and the GPU's pick must lie within the scoring tolerance of the oracle's minimum there; the
comparison then carries on from the GPU's state, so that one tolerated flip cannot cascade."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_14051_b200 as P

from parity import ATOL, RTOL, f32

pytestmark = pytest.mark.gpu
DEV = "cuda"


def follow(order_gpu, h, V, pos, k):
    """Returns the number of tolerated differences; raises on a pick outside the band."""
    n, d = V.shape
    remaining = list(range(n))
    t, flips = 0, 0
    while t < k:
        hr = h[remaining].astype(np.float64)
        o_order, _, _ = oracle.greedy_evict(hr / hr.sum(), V[remaining], k - t, pos[remaining])
        mapped = [remaining[i] for i in o_order]
        c = 0
        while c < k - t and mapped[c] == order_gpu[t + c]:
            c += 1
        if c == k - t:
            break
        gone = set(mapped[:c])
        rem2 = [j for j in remaining if j not in gone]
        r = oracle.score(np.zeros((1, 1, 1, d), np.float32), np.zeros((1, 1, len(rem2), d), np.float32), V[rem2][None, None],
                         np.array([len(rem2)], np.int32), scale=1.0, base_mode="external",
                         base=h[rem2][None, None].astype(np.float64))
        c_ref = r["scores"][0, 0]
        e = order_gpu[t + c]
        assert e in rem2, f"pick {t + c}: slot {e} was evicted before or is out of range"
        cmin = c_ref.min()
        assert abs(c_ref[rem2.index(e)] - cmin) <= ATOL + RTOL * abs(cmin), (
            f"pick {t + c}: GPU evicts slot {e} (oracle score {c_ref[rem2.index(e)]!r}) but the minimum is {cmin!r}")
        flips += 1
        remaining = [j for j in rem2 if j != e]
        t += c + 1
    return flips


@pytest.mark.parametrize("case", [
    # B, Hkv, d, cap, lens, k, dtype
    (2, 2, 128, 320, [300, 257], 2, torch.bfloat16),
    (2, 2, 128, 320, [300, 257], 8, torch.bfloat16),
    (1, 3, 64, 100, [97], 40, torch.float32),
    (1, 2, 128, 1300, [1280], 128, torch.bfloat16),     # a reduced prompt block: 1152 kept + 128 new, evict 128
    (1, 1, 128, 40, [33], 32, torch.bfloat16),          # down to a single token
    (2, 3, 128, 2104, [2000, 777], 64, torch.bfloat16), # the cluster kernel; the short sequence leaves most CTAs of its clusters without rows
    (1, 2, 128, 6160, [6150], 24, torch.bfloat16),      # the cluster kernel with several hundred rows per CTA
    (1, 2, 128, 13000, [12900], 24, torch.bfloat16),    # more rows than 16 CTAs hold in shared memory: the rest from L2
])
def test_greedy_sequence_follows_the_oracle(case):
    B, Hkv, d, cap, lens, k, dtype = case
    g = torch.Generator(device="cpu").manual_seed(k * 7 + d)
    V = torch.randn((B, Hkv, cap, d), generator=g).to(dtype)
    h = (torch.rand((B, Hkv, cap), generator=g) ** 3 + 1e-3).float()
    pos = torch.stack([torch.stack([torch.randperm(cap, generator=g) for _ in range(Hkv)]) for _ in range(B)]).to(torch.int32)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    budget = lens_t - k
    p = P.make_params(B, Hkv, Hkv, d, cap, 1, dtype, 1.0, "external")
    ws = P.alloc_workspace(p, DEV)
    ev = torch.full((B, Hkv, k), -1, dtype=torch.int32, device=DEV)
    order = torch.full((B, Hkv, k), -1, dtype=torch.int32, device=DEV)
    ne = torch.zeros((B,), dtype=torch.int32, device=DEV)
    P.caote_trace_enable(True)
    P.caote_select_evict_greedy(p, V.to(DEV), h.to(DEV), lens_t.to(DEV), budget.to(DEV), pos.to(DEV), ev, order, ne, ws)
    torch.cuda.synchronize()
    trace = P.caote_trace_collect()
    P.caote_trace_enable(False)
    assert P.caote_read_status(ws) == 0
    assert ne.cpu().tolist() == [k] * B
    if dtype == torch.bfloat16 and d == 128 and cap >= 1300:
        # long units with many picks: the kernel that keeps the value rows in the shared memory of a cluster
        assert "greedy_cluster_kernel" in trace, trace
    Vn, hn, pn = f32(V), h.numpy(), pos.numpy()
    flips = 0
    for b in range(B):
        n = lens[b]
        for hd in range(Hkv):
            og = order[b, hd].cpu().numpy().tolist()
            assert len(set(og)) == k and all(0 <= j < n for j in og)
            assert ev[b, hd].cpu().numpy().tolist() == sorted(og)
            flips += follow(og, hn[b, hd, :n], Vn[b, hd, :n], pn[b, hd, :n], k)
    assert flips <= max(1, (B * Hkv * k) // 20), f"{flips} tolerated differences: too many to be rounding"
    # a second run gives the same sequence
    order2 = torch.full_like(order, -1)
    P.caote_select_evict_greedy(p, V.to(DEV), h.to(DEV), lens_t.to(DEV), budget.to(DEV), pos.to(DEV), ev, order2, ne, ws)
    assert torch.equal(order, order2)


def test_one_greedy_pick_is_the_plain_selection_and_k0_evicts_nothing():
    B, Hkv, d, cap, n = 2, 2, 128, 700, 650
    g = torch.Generator(device="cpu").manual_seed(5)
    q = torch.randn((B, Hkv, 1, d), generator=g).to(torch.bfloat16).to(DEV)
    K = torch.randn((B, Hkv, cap, d), generator=g).to(torch.bfloat16).to(DEV)
    V = torch.randn((B, Hkv, cap, d), generator=g).to(torch.bfloat16).to(DEV)
    h = torch.rand((B, Hkv, cap), generator=g).to(DEV)
    lens = torch.tensor([n, n - 30], dtype=torch.int32, device=DEV)
    p = P.make_params(B, Hkv, Hkv, d, cap, 1, torch.bfloat16, d ** -0.5, "external")
    ws = P.alloc_workspace(p, DEV)
    o = torch.zeros((B, Hkv, 1, d), device=DEV)
    scores = torch.zeros((B, Hkv, cap), device=DEV)
    P.caote_score(p, q, K, V, lens, h, o, scores, ws)
    ev1 = torch.full((B, Hkv, 1), -1, dtype=torch.int32, device=DEV)
    ev2 = torch.full((B, Hkv, 1), -1, dtype=torch.int32, device=DEV)
    ne1 = torch.zeros((B,), dtype=torch.int32, device=DEV)
    ne2 = torch.zeros((B,), dtype=torch.int32, device=DEV)
    budget = lens - 1
    P.caote_select_evict(p, scores, lens, budget, None, ev1, ne1, ws)
    P.caote_select_evict_greedy(p, V, h, lens, budget, None, ev2, None, ne2, ws)
    sc = scores.cpu().numpy()
    for b in range(B):
        for hd in range(Hkv):
            a, c = int(ev1[b, hd, 0]), int(ev2[b, hd, 0])
            assert a == c or abs(sc[b, hd, a] - sc[b, hd, c]) <= ATOL + RTOL * sc[b, hd, a]
    assert ne1.tolist() == ne2.tolist() == [1, 1]
    P.caote_select_evict_greedy(p, V, h, lens, lens.clone(), None, ev2, None, ne2, ws)
    assert ne2.tolist() == [0, 0] and P.caote_read_status(ws) == 0
