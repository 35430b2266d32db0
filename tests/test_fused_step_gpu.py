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


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 64)])
@pytest.mark.parametrize("n", [300, 9000])
def test_equal_lowest_scores_go_by_position(dtype, d, n):
    """Three cached tokens of every unit are copies of one another (same key, same value) with by far the smallest
    weight, so their scores are the unit's lowest and, computed the same way, equal; positions are a permutation, so the
    copy in the highest slot can have the lowest position. The evicted slot is the arg-min over (score bits, position)
    of the scores this call wrote."""
    B, H, cap = 2, 2, n + 8
    c, q, vn, g = make_cache(B, H, d, n, cap, dtype, 300 + n)
    qf = q.float()
    low = (-(20.0 / (d ** -0.5 * (qf * qf).sum(-1, keepdim=True))) * qf).to(dtype)  # [B, H, 1, d]
    K0, V0 = c.K.clone(), c.V.clone()
    copies = [5, n // 2, n - 2]
    for j in copies:
        K0[:, :, j] = low[:, :, 0]
        V0[:, :, j] = V0[:, :, 5]
    pos0 = torch.stack([torch.stack([torch.randperm(cap, generator=g) for _ in range(H)]) for _ in range(B)]).to(torch.int32).to(DEV)
    c.load(K0, V0, torch.full((B,), n, dtype=torch.int32, device=DEV), pos=pos0)
    c.n_seen.fill_(cap)  # the new token's position: above every cached one
    kn = ((12.0 / (d ** -0.5 * (qf * qf).sum(-1, keepdim=True))) * qf).to(dtype)
    c.step(q, kn, vn)
    torch.cuda.synchronize()
    assert c.status() == 0 and c.n_evict.tolist() == [1] * B
    ties = 0
    for b in range(B):
        for h in range(H):
            sc = c.scores[b, h, :n + 1]
            cand = torch.nonzero(sc == sc.min()).flatten()
            ties += int(len(cand) > 1)
            pos_pre = torch.cat([pos0[b, h, :n], torch.tensor([cap], dtype=torch.int32, device=DEV)])
            want = int(cand[torch.argmin(pos_pre[cand])])
            assert int(c.evict_idx[b, h, 0]) == want
            assert want in copies
    assert ties > 0, "the copies' scores were expected to be equal in at least one unit"
