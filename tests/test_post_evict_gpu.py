"""Post-eviction attention output on the GPU (C ABI) against the oracle's definition: softmax attention over
the retained tokens, computed as a correction of the pre-eviction output."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_14051_b200 as P

from parity import assert_close, f32
from test_gpu_parity import make_case

pytestmark = pytest.mark.gpu
DEV = "cuda"

CASES = [
    # B, Hq, Hkv, d, cap, m, lens, budget, dtype
    (2, 8, 2, 128, 300, 1, [257, 129], [250, 100], torch.bfloat16),      # decode: evict 7 and 29
    (1, 7, 1, 128, 1100, 1, [1031], [1030], torch.bfloat16),             # evict 1
    (2, 4, 2, 64, 80, 1, [63, 80], [40, 80], torch.float32),             # one sequence evicts nothing
    (1, 8, 2, 128, 520, 128, [515], [387], torch.bfloat16),              # block of 128 queries, evict 128
    (2, 6, 2, 64, 96, 5, [90, 17], [60, 3], torch.float32),              # most of a short sequence goes
    (3, 32, 8, 128, 4224, 1, [4129, 515, 2000], [4096, 512, 2000], torch.bfloat16),  # several tiles per unit
    (1, 12, 2, 128, 700, 33, [640], [500], torch.bfloat16),              # ragged block, 6 heads per group
]
# cases whose scoring call runs on the tensor-core kernels and so leaves the rows' statistics in the workspace
LEAVES_STATS = {0, 1, 3, 5, 6}


@pytest.mark.parametrize("case", CASES)
def test_post_evict_output_matches_oracle(case):
    B, Hq, Hkv, d, cap, m, lens, budget, dtype = case
    q, K, V, lens_t = make_case(1234 + CASES.index(case), B, Hq, Hkv, d, cap, m, dtype, lens)
    mode = "last_query" if m == 1 else "chunk_sum"
    p = P.make_params(B, Hq, Hkv, d, cap, m, dtype, d ** -0.5, mode)
    ws = P.alloc_workspace(p, DEV)
    o = torch.zeros(q.shape, dtype=torch.float32, device=DEV)
    scores = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=DEV)
    P.caote_score(p, q, K, V, lens_t, None, o, scores, ws)
    max_evict = max(n - b for n, b in zip(lens, budget)) or 1
    evict_idx = torch.zeros((B, Hkv, max_evict), dtype=torch.int32, device=DEV)
    n_evict = torch.zeros((B,), dtype=torch.int32, device=DEV)
    budget_t = torch.tensor(budget, dtype=torch.int32, device=DEV)
    P.caote_select_evict(p, scores, lens_t, budget_t, None, evict_idx, n_evict, ws)
    o_post = torch.full_like(o, float("nan"))
    P.caote_post_evict_output(p, q, K, V, lens_t, evict_idx, n_evict, o, o_post)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    ne, ev = n_evict.cpu().numpy(), evict_idx.cpu().numpy()
    evict = [[ev[b, h, :ne[b]] for h in range(Hkv)] for b in range(B)]
    ref = oracle.post_evict_output(f32(q), f32(K), f32(V), lens, evict, scale=d ** -0.5, n_new=m)
    got = f32(o_post)
    for b in range(B):
        assert ne[b] == max(0, lens[b] - budget[b])
        assert_close(got[b], ref[b], f"{case} o_post[b={b}]")
        if ne[b] == 0:
            assert_close(got[b], f32(o)[b], "nothing evicted: the output is unchanged", rtol=1e-6, atol=1e-7)
    # in place
    o2 = o.clone()
    P.caote_post_evict_output(p, q, K, V, lens_t, evict_idx, n_evict, o2, o2)
    torch.cuda.synchronize()
    assert torch.equal(o2, o_post)
    # from the statistics the scoring call left in the workspace
    o3 = torch.full_like(o, float("nan"))
    K3 = K
    if CASES.index(case) in LEAVES_STATS:
        # the statistics stand in for the pass over K: only the evicted rows of K may be read, so every other row
        # can hold anything (a pass over K would turn the result into NaN)
        K3 = torch.full_like(K, float("nan"))
        for b in range(B):
            for h in range(Hkv):
                idx = torch.as_tensor(np.asarray(evict[b][h], dtype=np.int64), device=DEV)
                K3[b, h, idx] = K[b, h, idx]
    P.caote_post_evict_output_ws(p, q, K3, V, lens_t, evict_idx, n_evict, o, o3, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    got3 = f32(o3)
    for b in range(B):
        assert_close(got3[b], ref[b], f"{case} o_post from the workspace statistics [b={b}]")


def test_statistics_of_another_scoring_path_are_not_used():
    """A tensor-core scoring call followed, on the same workspace, by one on the any-shape path: the second call
    marks the workspace as holding no statistics and the post-eviction output falls back to its pass over K."""
    B, Hq, Hkv, d, cap, dtype = 1, 8, 2, 128, 300, torch.bfloat16
    lens, budget = [257], [250]
    q, K, V, lens_t = make_case(77, B, Hq, Hkv, d, cap, 1, dtype, lens)
    p1 = P.make_params(B, Hq, Hkv, d, cap, 1, dtype, d ** -0.5, "last_query")
    ws = P.alloc_workspace(p1, DEV)
    o = torch.zeros(q.shape, dtype=torch.float32, device=DEV)
    scores = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=DEV)
    P.caote_score(p1, q, K, V, lens_t, None, o, scores, ws)          # cluster kernel: leaves statistics
    P.caote_set_option(P.OPT_DECODE_CLUSTER, -1)
    try:
        scale = 0.5 * d ** -0.5                                       # other logits: the old statistics would be wrong
        p2 = P.make_params(B, Hq, Hkv, d, cap, 1, dtype, scale, "last_query")
        P.caote_score(p2, q, K, V, lens_t, None, o, scores, ws)      # streaming kernel: leaves none
    finally:
        P.caote_set_option(P.OPT_DECODE_CLUSTER, 0)
    evict_idx = torch.zeros((B, Hkv, 7), dtype=torch.int32, device=DEV)
    n_evict = torch.zeros((B,), dtype=torch.int32, device=DEV)
    P.caote_select_evict(p2, scores, lens_t, torch.tensor(budget, dtype=torch.int32, device=DEV), None, evict_idx, n_evict, ws)
    o_post = torch.full_like(o, float("nan"))
    P.caote_post_evict_output_ws(p2, q, K, V, lens_t, evict_idx, n_evict, o, o_post, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    ev = evict_idx.cpu().numpy()
    ref = oracle.post_evict_output(f32(q), f32(K), f32(V), lens, [[ev[0, h] for h in range(Hkv)]], scale=scale, n_new=1)
    assert_close(f32(o_post)[0], ref[0], "fallback to the pass over K")
