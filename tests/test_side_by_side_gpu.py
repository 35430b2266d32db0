"""Single-query scoring with the cluster kernel and the streaming kernel side by side (the last sequences of the
batch on a second stream): results against the oracle for every unit, the statistics both kernels leave for the
post-eviction output, and the same call with the option off."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_14051_b200 as P

from parity import assert_close, check_scores_and_o, f32, oracle_for
from test_gpu_parity import make_case

pytestmark = pytest.mark.gpu
DEV = "cuda"

# (the library takes this route by itself only where its estimate says it pays, e.g. the 64 units of 16 385 tokens of
# the long-context decode workload; here the option forces it on a small case: the last sequence's four units go to the
# streaming kernel, the other twelve to the cluster kernel)
B, HQ, HKV, D, CAP = 4, 16, 4, 128, 1152
LENS = [1100, 900, 1152, 700]


def score(mode, side_by_side, base=None):
    q, K, V, lens_t = make_case(4242, B, HQ, HKV, D, CAP, 1, torch.bfloat16, LENS)
    p = P.make_params(B, HQ, HKV, D, CAP, 1, torch.bfloat16, D ** -0.5, mode)
    ws = P.alloc_workspace(p, DEV)
    o = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    scores = torch.full((B, HKV, CAP), -7.0, dtype=torch.float32, device=DEV)
    P.caote_set_option(P.OPT_SIDE_BY_SIDE, 2 if side_by_side else 0)
    P.caote_trace_enable(True)
    try:
        P.caote_score(p, q, K, V, lens_t, base, o, scores, ws)
        torch.cuda.synchronize()
    finally:
        P.caote_set_option(P.OPT_SIDE_BY_SIDE, 1)
        trace = P.caote_trace_collect()
        P.caote_trace_enable(False)
    assert P.caote_read_status(ws) == 0
    return p, ws, q, K, V, lens_t, o, scores, trace


@pytest.mark.parametrize("mode", ["last_query", "accum"])
def test_side_by_side_matches_the_oracle_and_the_single_kernel(mode):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(5)
    base0 = torch.rand((B, HKV, CAP), device=DEV, generator=gen) if mode == "accum" else None
    base = None if base0 is None else base0.clone()
    p, ws, q, K, V, lens_t, o, scores, trace = score(mode, True, base)
    assert "decode_side_by_side" in trace and "decode_tc_kernel" in trace and "decode_cluster_kernel" in trace, trace
    r = oracle_for(q, K, V, lens_t, scale=D ** -0.5, n_new=1, base_mode=mode, base=base0)
    check_scores_and_o(r, scores, o, lens_t, f"side by side {mode}")
    if mode == "accum":  # the carried scores are updated in place by both kernels
        for b, n in enumerate(LENS):
            assert_close(f32(base)[b, :, :n], r["base"][b, :, :n], f"carried base scores [b={b}]")
    # the option off: one kernel, same results within the tolerance of either
    base1 = None if base0 is None else base0.clone()
    _, _, _, _, _, _, o1, scores1, trace1 = score(mode, False, base1)
    assert "decode_side_by_side" not in trace1 and "decode_tc_kernel" not in trace1, trace1
    check_scores_and_o(r, scores1, o1, lens_t, f"single kernel {mode}")

    # both kernels leave the heads' log-sum-exp: the post-eviction output needs no pass over K for any unit
    budget = torch.tensor([n - 3 for n in LENS], dtype=torch.int32, device=DEV)
    evict_idx = torch.zeros((B, HKV, 3), dtype=torch.int32, device=DEV)
    n_evict = torch.zeros((B,), dtype=torch.int32, device=DEV)
    P.caote_select_evict(p, scores, lens_t, budget, None, evict_idx, n_evict, ws)
    torch.cuda.synchronize()
    ev = evict_idx.cpu().numpy()
    K3 = torch.full_like(K, float("nan"))
    for b in range(B):
        for h in range(HKV):
            idx = torch.as_tensor(ev[b, h].astype(np.int64), device=DEV)
            K3[b, h, idx] = K[b, h, idx]
    o_post = torch.full_like(o, float("nan"))
    P.caote_post_evict_output_ws(p, q, K3, V, lens_t, evict_idx, n_evict, o, o_post, ws)
    torch.cuda.synchronize()
    assert P.caote_read_status(ws) == 0
    ref = oracle.post_evict_output(f32(q), f32(K), f32(V), LENS, [[ev[b, h] for h in range(HKV)] for b in range(B)],
                                   scale=D ** -0.5, n_new=1)
    for b in range(B):
        assert_close(f32(o_post)[b], ref[b], f"post-eviction output from the statistics [b={b}]")


def test_side_by_side_with_empty_sequences():
    """An empty sequence among those of the cluster kernel and an empty one as the streaming kernel's whole share:
    their outputs are left alone, the others match the oracle."""
    lens = [1100, 0, 1152, 0]
    q, K, V, lens_t = make_case(777, B, HQ, HKV, D, CAP, 1, torch.bfloat16, lens)
    p = P.make_params(B, HQ, HKV, D, CAP, 1, torch.bfloat16, D ** -0.5, "last_query")
    ws = P.alloc_workspace(p, DEV)
    o = torch.full(q.shape, -3.0, dtype=torch.float32, device=DEV)
    scores = torch.full((B, HKV, CAP), -7.0, dtype=torch.float32, device=DEV)
    P.caote_set_option(P.OPT_SIDE_BY_SIDE, 2)
    try:
        P.caote_score(p, q, K, V, lens_t, None, o, scores, ws)
        torch.cuda.synchronize()
    finally:
        P.caote_set_option(P.OPT_SIDE_BY_SIDE, 1)
    assert P.caote_read_status(ws) == 0
    r = oracle_for(q, K, V, lens_t, scale=D ** -0.5, n_new=1, base_mode="last_query")
    check_scores_and_o(r, scores, o, lens_t, "side by side, empty sequences")
    for b in (1, 3):
        assert (f32(scores)[b] == -7.0).all() and (f32(o)[b] == -3.0).all()
