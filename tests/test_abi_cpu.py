"""CPU-side checks of the C ABI: the library loads, exports what the header declares, and rejects
bad arguments on the host before touching a device. No compute call is made here."""
import ctypes
import os
import re

import pytest
import torch

import paper_2504_14051_b200 as P
from paper_2504_14051_b200 import binding as C

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"CAOTE_API\s+[\w\s\*]+?\b(caote_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol():
    lib = P.lib()
    names = declared_symbols()
    assert {"caote_score", "caote_select_evict", "caote_compact", "caote_append", "caote_step",
            "caote_workspace_bytes", "caote_read_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"


def test_params_struct_matches_header():
    text = open(os.path.join(ROOT, "include", "caote.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} caote_params_t;", text, re.S).group(1)
    fields = re.findall(r"^\s*(int32_t|float)\s+(\w+);", body, re.M)
    assert [f for _, f in fields] == [f for f, _ in C.Params._fields_]
    assert ctypes.sizeof(C.Params) == 4 * len(fields)


def test_status_strings_and_workspace_size():
    for code in range(0, -8, -1):
        assert C.caote_status_string(code) != "unknown status"
    assert C.caote_status_string(-99) == "unknown status"
    p = C.make_params(2, 8, 2, 128, 1024, 1, torch.bfloat16, 0.1, "accum")
    n1 = C.caote_workspace_bytes(p)
    assert n1 > 256
    p2 = C.make_params(2, 8, 2, 128, 1024, 128, torch.bfloat16, 0.1, "chunk_sum")
    assert C.caote_workspace_bytes(p2) > n1
    # invalid or unsupported parameters give 0
    for bad in [C.make_params(0, 8, 2, 128, 16, 1, 0, 0.1, 0), C.make_params(1, 7, 2, 128, 16, 1, 0, 0.1, 0),
                C.make_params(1, 8, 2, 96, 16, 1, 0, 0.1, 0), C.make_params(1, 8, 2, 128, 16, 1, 5, 0.1, 0),
                C.make_params(1, 8, 2, 128, 16, 17, 0, 0.1, 0), C.make_params(1, 34, 2, 128, 16, 1, 0, 0.1, 0),
                C.make_params(1, 8, 2, 128, 16, 1, 0, 0.1, 4)]:
        assert C.caote_workspace_bytes(bad) == 0


def test_host_side_argument_checks_return_before_any_launch():
    lib = P.lib()
    before = C.caote_launch_count()
    p = C.make_params(1, 4, 2, 64, 32, 1, torch.float32, 0.125, "accum")
    need = C.caote_workspace_bytes(p)
    fake = ctypes.c_void_p(4096)  # never dereferenced: validation fails first
    ws = ctypes.c_void_p(1 << 20)
    bp = ctypes.byref(p)
    # null pointers
    assert lib.caote_score(bp, None, fake, fake, fake, fake, fake, fake, ws, need, None) == C.ERR_INVALID_ARG
    # accum needs base
    assert lib.caote_score(bp, fake, fake, fake, fake, None, fake, fake, ws, need, None) == C.ERR_INVALID_ARG
    # workspace too small / misaligned
    assert lib.caote_score(bp, fake, fake, fake, fake, fake, fake, fake, ws, need - 1, None) == C.ERR_INVALID_ARG
    assert lib.caote_score(bp, fake, fake, fake, fake, fake, fake, fake, ctypes.c_void_p((1 << 20) + 8), need,
                           None) == C.ERR_INVALID_ARG
    # misaligned K
    assert lib.caote_score(bp, fake, ctypes.c_void_p(4100), fake, fake, fake, fake, fake, ws, need,
                           None) == C.ERR_INVALID_ARG
    # unsupported head_dim
    p96 = C.make_params(1, 4, 2, 96, 32, 1, torch.float32, 0.125, "last_query")
    assert lib.caote_score(ctypes.byref(p96), fake, fake, fake, fake, fake, fake, fake, ws, 1 << 20,
                           None) == C.ERR_UNSUPPORTED
    assert lib.caote_select_evict(bp, fake, fake, fake, None, fake, 0, fake, ws, need, None) == C.ERR_INVALID_ARG
    assert lib.caote_compact(bp, fake, fake, None, None, fake, fake, 4, fake, 7, ws, need, None) == C.ERR_INVALID_ARG
    assert lib.caote_append(bp, fake, fake, None, None, None, None, fake, fake, ws, need, None) == C.ERR_INVALID_ARG
    assert lib.caote_read_status(None, None, None) == C.ERR_INVALID_ARG
    # FastCAOTE entry points: the running sum of value rows is mandatory and 16-byte aligned
    assert lib.caote_vsum(bp, fake, fake, None, None) == C.ERR_INVALID_ARG
    assert lib.caote_vsum(None, fake, fake, fake, None) == C.ERR_INVALID_ARG
    assert lib.caote_score_fast(bp, fake, fake, fake, fake, fake, None, fake, fake, ws, need, None) == C.ERR_INVALID_ARG
    assert lib.caote_score_fast(bp, fake, fake, fake, fake, fake, ctypes.c_void_p(4100), fake, fake, ws, need,
                                None) == C.ERR_INVALID_ARG
    assert lib.caote_score_fast(bp, fake, fake, fake, fake, fake, fake, fake, fake, ws, need - 1, None) == C.ERR_INVALID_ARG
    assert lib.caote_step_fast(bp, fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, None, fake, fake, fake, 1,
                               fake, 0, ws, need, None) == C.ERR_INVALID_ARG
    # sum-of-errors aggregation: defined for LAST_QUERY and CHUNK_SUM only (p is ACCUM)
    assert lib.caote_score_sum_errors(bp, fake, fake, fake, fake, fake, fake, ws, need, None) == C.ERR_UNSUPPORTED
    assert lib.caote_score_sum_errors(bp, None, fake, fake, fake, fake, fake, ws, need, None) == C.ERR_INVALID_ARG
    # post-eviction output: every pointer is mandatory, max_evict >= 1
    assert lib.caote_post_evict_output(bp, fake, fake, fake, fake, None, 4, fake, fake, fake, None) == C.ERR_INVALID_ARG
    assert lib.caote_post_evict_output(bp, fake, fake, fake, fake, fake, 0, fake, fake, fake, None) == C.ERR_INVALID_ARG
    assert lib.caote_post_evict_output(bp, fake, fake, fake, fake, fake, 4, fake, fake, None, None) == C.ERR_INVALID_ARG
    # ... and the variant that reuses the scoring call's statistics also wants that call's workspace
    assert lib.caote_post_evict_output_ws(bp, fake, fake, fake, fake, fake, 4, fake, fake, fake, None, need, None) == C.ERR_INVALID_ARG
    assert lib.caote_post_evict_output_ws(bp, fake, fake, fake, fake, fake, 4, fake, fake, fake, ws, need - 1, None) == C.ERR_INVALID_ARG
    assert lib.caote_post_evict_output_ws(bp, fake, fake, fake, fake, fake, 4, fake, fake, fake, ctypes.c_void_p(4100), need,
                                          None) == C.ERR_INVALID_ARG
    assert lib.caote_post_evict_output_ws(bp, fake, fake, fake, fake, None, 4, fake, fake, fake, ws, need, None) == C.ERR_INVALID_ARG
    # the whole-step entry points validate append, score and selection arguments before their first launch
    # (the FastCAOTE step would otherwise have added the new rows to the running sum already)
    okp = C.make_params(1, 4, 2, 64, 32, 1, torch.float32, 0.125, "last_query")
    okb, okneed = ctypes.byref(okp), C.caote_workspace_bytes(okp)
    for bad_K in (None, ctypes.c_void_p(4100)):
        assert lib.caote_step_fast(okb, fake, fake, fake, bad_K, fake, None, fake, fake, fake, fake, fake, fake, fake, fake,
                                   1, fake, 0, ws, okneed, None) == C.ERR_INVALID_ARG
        assert lib.caote_step(okb, fake, fake, fake, bad_K, fake, None, fake, fake, fake, fake, fake, fake, fake, 1, fake,
                              0, ws, okneed, None) == C.ERR_INVALID_ARG
    assert lib.caote_step_fast(okb, fake, fake, fake, fake, fake, None, fake, fake, fake, fake, fake, fake, fake, fake, 1,
                               fake, 0, ws, okneed - 1, None) == C.ERR_INVALID_ARG          # workspace too small
    assert lib.caote_step_fast(okb, fake, fake, fake, fake, fake, None, fake, fake, fake, None, fake, fake, fake, fake, 1,
                               fake, 0, ws, okneed, None) == C.ERR_INVALID_ARG              # no budget
    assert lib.caote_step_fast(ctypes.byref(p96), fake, fake, fake, fake, fake, None, fake, fake, fake, fake, fake, fake,
                               fake, fake, 1, fake, 0, ws, 1 << 20, None) == C.ERR_UNSUPPORTED
    # the no-allocation variant refuses what caote_score refuses, before it touches its built-in array
    assert lib.caote_score_static(okb, None, fake, fake, fake, None, fake, fake, None, None) == C.ERR_INVALID_ARG
    assert lib.caote_score_static(okb, fake, ctypes.c_void_p(4100), fake, fake, None, fake, fake, None, None) == C.ERR_INVALID_ARG
    assert lib.caote_score_static(bp, fake, fake, fake, fake, None, fake, fake, None, None) == C.ERR_INVALID_ARG  # accum, no base
    big = C.make_params(64, 28, 4, 128, 8196, 1, torch.bfloat16, 0.1, "accum")
    assert lib.caote_score_static(ctypes.byref(big), fake, fake, fake, fake, fake, fake, fake, None, None) == C.ERR_TOO_LARGE
    assert C.caote_launch_count() == before


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a box without a GPU")
def test_product_path_fails_loudly_without_a_gpu():
    p = C.make_params(1, 4, 2, 64, 32, 1, torch.float32, 0.125, "last_query")
    need = C.caote_workspace_bytes(p)
    fake, ws = ctypes.c_void_p(4096), ctypes.c_void_p(1 << 20)
    rc = P.lib().caote_score(ctypes.byref(p), fake, fake, fake, fake, None, fake, fake, ws, need, None)
    assert rc in (C.ERR_CUDA, C.ERR_UNSUPPORTED)  # no device: an error, never a silent CPU result
