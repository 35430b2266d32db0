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
]


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
