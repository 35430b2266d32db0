"""The sum-of-errors aggregation on the GPU against the oracle (agg_mode="sum_errors")."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_14051_b200 as P

from parity import assert_close, f32
from test_gpu_parity import dominant_case, make_case

pytestmark = pytest.mark.gpu
DEV = "cuda"

CASES = [
    # B, Hq, Hkv, d, cap, m, lens, dtype, mode
    (1, 1, 1, 64, 40, 1, [37], torch.float32, "last_query"),          # one head, one query: equals caote_score
    (2, 8, 2, 128, 300, 1, [257, 129], torch.bfloat16, "last_query"),
    (2, 4, 2, 64, 80, 1, [63, 0], torch.float32, "last_query"),
    (1, 14, 2, 128, 400, 3, [333], torch.bfloat16, "chunk_sum"),
    (2, 8, 4, 64, 272, 40, [272, 130], torch.bfloat16, "chunk_sum"),
    (1, 6, 2, 128, 200, 5, [5], torch.float32, "last_query"),         # only the new block is cached
    # one query per head in bf16 / d 128: the cluster kernel, then the pass of sum_errors_decode.cuh
    (2, 28, 4, 128, 1300, 1, [1290, 515], torch.bfloat16, "last_query"),   # 7 heads per group, ragged tiles
    (1, 64, 8, 128, 2100, 1, [2049], torch.bfloat16, "chunk_sum"),         # 8 heads per group, one token in the last tile
    (3, 2, 2, 128, 144, 1, [1, 0, 129], torch.bfloat16, "last_query"),     # a single cached token; an empty sequence
]


@pytest.mark.parametrize("case", CASES)
def test_sum_errors_scores_match_oracle(case):
    B, Hq, Hkv, d, cap, m, lens, dtype, mode = case
    q, K, V, lens_t = make_case(555 + CASES.index(case), B, Hq, Hkv, d, cap, m, dtype, lens)
    p = P.make_params(B, Hq, Hkv, d, cap, m, dtype, d ** -0.5, mode)
    ws = P.alloc_workspace(p, DEV)
    o = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    scores = torch.full((B, Hkv, cap), -7.0, dtype=torch.float32, device=DEV)
    P.caote_score_sum_errors(p, q, K, V, lens_t, o, scores, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    r = oracle.score(f32(q), f32(K), f32(V), lens_t.cpu().numpy(), scale=d ** -0.5, n_new=m, base_mode=mode,
                     agg_mode="sum_errors")
    sg, og = f32(scores), f32(o)
    for b, n in enumerate(lens):
        if n == 0:
            continue
        assert_close(sg[b, :, :n], r["scores"][b, :, :n], f"{case} sum-of-errors scores[b={b}]")
        assert (sg[b, :, n:] == -7.0).all()
        assert_close(og[b], r["o"][b], f"{case} o[b={b}]")
    if Hq == 1 and m == 1:
        ref = torch.zeros_like(scores)
        P.caote_score(p, q, K, V, lens_t, None, o, ref, ws)
        torch.cuda.synchronize()
        assert_close(sg[0, 0, :lens[0]], f32(ref)[0, 0, :lens[0]], "one head, one query: both aggregations agree", rtol=1e-4)


def test_sum_errors_refuses_carried_base_modes():
    p = P.make_params(1, 4, 2, 64, 32, 1, torch.float32, 0.125, "accum")
    ws = P.alloc_workspace(p, DEV)
    t = torch.zeros(8, device=DEV)
    with pytest.raises(P.CaoteError):
        P.caote_score_sum_errors(p, t, t, t, torch.zeros(1, dtype=torch.int32, device=DEV), t, t, ws)


@pytest.mark.parametrize("eps", [1e-1, 1e-3])
def test_sum_errors_with_a_token_that_holds_almost_all_the_weight(eps):
    """Single-query path: 1 - alpha of the planted token is the stored share of the others (about eps), not a
    difference of nearly equal numbers."""
    B, Hq, Hkv, d, cap, lens = 2, 8, 2, 128, 1600, [1531, 700]
    q, K, V, lens_t = dominant_case(911, B, Hq, Hkv, d, cap, 1, torch.bfloat16, lens, eps, 77)
    p = P.make_params(B, Hq, Hkv, d, cap, 1, torch.bfloat16, d ** -0.5, "last_query")
    ws = P.alloc_workspace(p, DEV)
    o = torch.zeros(q.shape, dtype=torch.float32, device=DEV)
    scores = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=DEV)
    P.caote_score_sum_errors(p, q, K, V, lens_t, o, scores, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    r = oracle.score(f32(q), f32(K), f32(V), lens_t.cpu().numpy(), scale=d ** -0.5, n_new=1, base_mode="last_query",
                     agg_mode="sum_errors")
    assert (1.0 - r["alpha_max"] < 3 * eps).all() if "alpha_max" in r else True
    for b, n in enumerate(lens):
        assert_close(f32(scores)[b, :, :n], r["scores"][b, :, :n], f"eps {eps} sum-of-errors scores[b={b}]")
