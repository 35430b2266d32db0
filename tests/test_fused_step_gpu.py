"""The fused step (append, score, select + FILL compaction in one call) on the cases its single-eviction path has of
its own: the token to evict is the unit's last row (nothing moves), or any other row (the last row fills the hole),
checked on the cache contents, not only on the indices."""
import pytest
import torch

import paper_2504_14051_b200 as P

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_cache(B, H, d, n, cap, dtype, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    c = P.EvictionCache(B, H, H, d, cap, 1, dtype, n, "last_query", "fill", d ** -0.5, max_evict=1, device=DEV)
    K0 = torch.randn((B, H, cap, d), generator=g).to(dtype).to(DEV)
    V0 = torch.randn((B, H, cap, d), generator=g).to(dtype).to(DEV)
    c.load(K0, V0, torch.full((B,), n, dtype=torch.int32, device=DEV))
    q = torch.randn((B, H, 1, d), generator=g).to(dtype).to(DEV)
    vn = torch.randn((B, H, 1, d), generator=g).to(dtype).to(DEV)
    return c, q, vn, g


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 64), (torch.float32, 128)])
@pytest.mark.parametrize("n", [37, 2049, 9000])
def test_new_token_with_the_lowest_score_is_evicted_in_place(dtype, d, n):
    """One head per unit; the new key points away from the query (logit -20 below zero), so the new token has by far
    the smallest weight and score: it is the unit's last row, which is evicted without a move."""
    B, H, cap = 3, 2, n + 8
    c, q, vn, _ = make_cache(B, H, d, n, cap, dtype, 100 + n)
    qf = q.float()
    kn = (-(20.0 / (d ** -0.5 * (qf * qf).sum(-1, keepdim=True))) * qf).to(dtype)
    K0, V0, pos0 = c.K.clone(), c.V.clone(), c.pos.clone()
    c.step(q, kn, vn)
    torch.cuda.synchronize()
    assert c.status() == 0
    assert c.n_evict.tolist() == [1] * B and c.lens.tolist() == [n] * B
    assert (c.evict_idx[:, :, 0] == n).all()
    assert torch.equal(c.K[:, :, :n], K0[:, :, :n]) and torch.equal(c.V[:, :, :n], V0[:, :, :n])
    assert torch.equal(c.pos[:, :, :n], pos0[:, :, :n])


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 64), (torch.float32, 128)])
@pytest.mark.parametrize("n", [37, 2049, 9000])
def test_last_row_fills_the_hole(dtype, d, n):
    """The new key is the query's direction (the largest weight by far), so some older token goes: the new token's row
    lands in its slot, every other row stays where it was."""
    B, H, cap = 3, 2, n + 8
    c, q, vn, _ = make_cache(B, H, d, n, cap, dtype, 200 + n)
    qf = q.float()
    kn = ((12.0 / (d ** -0.5 * (qf * qf).sum(-1, keepdim=True))) * qf).to(dtype)
    K0, V0, pos0 = c.K.clone(), c.V.clone(), c.pos.clone()
    c.step(q, kn, vn)
    torch.cuda.synchronize()
    assert c.status() == 0
    assert c.n_evict.tolist() == [1] * B and c.lens.tolist() == [n] * B
    scores = c.scores.clone()
    for b in range(B):
        for h in range(H):
            e = int(c.evict_idx[b, h, 0])
            assert 0 <= e < n
            # the evicted slot is the argmin of the scores this call wrote (ties: the lower position)
            sc = scores[b, h, :n + 1]
            assert float(sc[e]) == float(sc.min())
            assert e == int(torch.nonzero(sc == sc.min())[0])
            keep = torch.ones(n, dtype=torch.bool, device=DEV)
            keep[e] = False
            assert torch.equal(c.K[b, h, :n][keep], K0[b, h, :n][keep])
            assert torch.equal(c.V[b, h, :n][keep], V0[b, h, :n][keep])
            assert torch.equal(c.K[b, h, e], kn[b, h, 0]) and torch.equal(c.V[b, h, e], vn[b, h, 0])
            assert int(c.pos[b, h, e]) == n and torch.equal(c.pos[b, h, :n][keep], pos0[b, h, :n][keep])
