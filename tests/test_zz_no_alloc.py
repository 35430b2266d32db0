"""caote_score_static: the scoring call for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: a serving engine whose memory pool
already owns the whole GPU, a plug-in that is handed tensors but no allocator, a latency path where
an allocation could stall the device. They cannot supply the workspace that caote_score wants, so
caote_score_static takes none and works on a fixed array inside the library instead.

Checked here, through the C ABI: the same inputs give the same outputs as caote_score and as the CPU
oracle, on two calls in a row (the array is shared and keeps the previous call's contents, so the
second call runs on a dirty array), for shapes served by the single-query kernel, by the tensor-core
kernels for a block of queries and by the any-shape kernels; the amount of device memory in use does not
move across a call; and a shape whose scratch would not fit the array is refused before anything runs.

This file sorts last on purpose, so a run that stops at the first failure has already run the rest.
"""
import ctypes

import pytest
import torch

import paper_2504_14051_b200 as P
from paper_2504_14051_b200 import binding as C

from parity import ATOL, RTOL, assert_close, check_scores_and_o, f32, oracle_for

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(seed, B, Hq, Hkv, d, cap, m, lens):
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn((B, Hq, m, d), generator=g).to(torch.bfloat16).to(DEV)
    K = torch.randn((B, Hkv, cap, d), generator=g).to(torch.bfloat16).to(DEV)
    V = torch.randn((B, Hkv, cap, d), generator=g).to(torch.bfloat16).to(DEV)
    base = (torch.rand((B, Hkv, cap), generator=g) * 3.0).to(DEV)
    return q, K, V, base, torch.tensor(lens, dtype=torch.int32, device=DEV)


@pytest.mark.parametrize("shape,mode", [
    ((3, 14, 2, 128, 1500, 1, [1500, 1031, 77]), "accum"),       # single-query kernel, carried base score
    ((2, 8, 2, 128, 700, 1, [700, 513]), "last_query"),          # single-query kernel
    ((1, 8, 2, 128, 400, 64, [390]), "chunk_sum"),               # tensor-core kernels for a block of 64 queries
    ((1, 4, 2, 64, 300, 3, [290]), "chunk_sum"),                 # any-shape kernels (head_dim 64, 3 queries)
])
def test_static_scratch_matches_workspace_call_twice(shape, mode):
    B, Hq, Hkv, d, cap, m, lens = shape
    q, K, V, base0, lens_t = _inputs(31, B, Hq, Hkv, d, cap, m, lens)
    p = P.make_params(B, Hq, Hkv, d, cap, m, torch.bfloat16, d ** -0.5, mode)
    assert 0 < P.caote_workspace_bytes(p) <= C.STATIC_SCRATCH_BYTES

    def outputs():
        return (torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV),
                torch.full((B, Hkv, cap), -3.0, dtype=torch.float32, device=DEV))

    # the existing entry point, on a workspace the caller allocated
    ws = P.alloc_workspace(p, DEV)
    o_ref, sc_ref = outputs()
    base_ref = base0.clone()
    P.caote_score(p, q, K, V, lens_t, base_ref if mode == "accum" else None, o_ref, sc_ref, ws)
    assert P.caote_read_status(ws) == 0

    r = oracle_for(q, K, V, lens_t, scale=d ** -0.5, n_new=m, base_mode=mode, base=base0 if mode == "accum" else None)
    for call in range(2):
        o, sc = outputs()
        base = base0.clone()
        status = torch.full((1,), 99, dtype=torch.int32, device=DEV)
        torch.cuda.synchronize()
        free_before, in_use_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        P.caote_score_static(p, q, K, V, lens_t, base if mode == "accum" else None, o, sc, status)
        torch.cuda.synchronize()
        # nothing was allocated or freed on the device by the call (neither through torch nor behind its back)
        assert torch.cuda.memory_allocated() == in_use_before and torch.cuda.mem_get_info()[0] == free_before
        assert status.item() == 0, f"call {call}: device status {status.item()}"
        check_scores_and_o(r, sc, o, lens_t, f"{shape} {mode} call {call} against the oracle")
        what = f"{shape} {mode} call {call}"
        assert_close(f32(sc), f32(sc_ref), what + " scores", rtol=RTOL, atol=ATOL)
        assert_close(f32(o)[[b for b, n in enumerate(lens) if n > 0]],
                     f32(o_ref)[[b for b, n in enumerate(lens) if n > 0]], what + " o", rtol=RTOL, atol=ATOL)
        if mode == "accum":
            assert_close(f32(base), f32(base_ref), what + " base", rtol=RTOL, atol=ATOL)


def test_static_scratch_reports_device_side_errors_and_refuses_oversize():
    B, Hq, Hkv, d, cap, m = 1, 8, 2, 128, 300, 1
    q, K, V, _, _ = _inputs(5, B, Hq, Hkv, d, cap, m, [300])
    p = P.make_params(B, Hq, Hkv, d, cap, m, torch.bfloat16, d ** -0.5, "last_query")
    o = torch.zeros(q.shape, dtype=torch.float32, device=DEV)
    sc = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=DEV)
    status = torch.zeros((1,), dtype=torch.int32, device=DEV)
    bad_len = torch.tensor([cap + 1], dtype=torch.int32, device=DEV)  # the kernel skips it and says so
    P.caote_score_static(p, q, K, V, bad_len, None, o, sc, status)
    torch.cuda.synchronize()
    assert status.item() == C.ERR_BAD_LENGTH
    # the next call starts from a clean status word
    P.caote_score_static(p, q, K, V, torch.tensor([cap], dtype=torch.int32, device=DEV), None, o, sc, status)
    torch.cuda.synchronize()
    assert status.item() == 0

    # a shape whose scratch exceeds the built-in array: refused on the host, nothing enqueued
    big = P.make_params(64, 32, 8, 128, 16384, 1, torch.bfloat16, d ** -0.5, "last_query")
    assert P.caote_workspace_bytes(big) > C.STATIC_SCRATCH_BYTES
    before = P.caote_launch_count()
    fake = ctypes.c_void_p(4096)  # never dereferenced
    rc = P.lib().caote_score_static(ctypes.byref(big), fake, fake, fake, fake, None, fake, fake, None, None)
    assert rc == C.ERR_TOO_LARGE and "scratch" in P.caote_status_string(rc)
    assert P.caote_launch_count() == before
