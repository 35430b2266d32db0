"""Helpers shared by the GPU parity tests: run the oracle on the same bits and compare.

Tolerances (bf16 or fp32 inputs, fp32 accumulation on the GPU, fp64 in the oracle):
scores and attention outputs  |gpu - ref| <= 1e-5 + 2e-3 * |ref|;
evicted sets identical except for tokens whose oracle score lies within that tolerance of the
selection threshold (the oracle's k-th smallest score).
"""
from __future__ import annotations

import numpy as np
import torch

import oracle

RTOL, ATOL = 2e-3, 1e-5


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def assert_close(gpu: np.ndarray, ref: np.ndarray, what: str, rtol=RTOL, atol=ATOL):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    both_inf = np.isinf(gpu) & np.isinf(ref) & (np.sign(gpu) == np.sign(ref))
    with np.errstate(invalid="ignore"):
        err = np.abs(np.where(both_inf, 0.0, gpu - ref))
    tol = atol + rtol * np.abs(np.where(both_inf, 0.0, ref))
    bad = ~(err <= tol)
    if bad.any():
        i = np.unravel_index(np.argmax(np.where(bad, err - tol, -np.inf)), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: "
                             f"gpu={gpu[i]!r} ref={ref[i]!r}")


def oracle_for(q, K, V, lens, *, scale, n_new, base_mode, base=None):
    """Run the oracle on the exact values held by torch tensors (any device)."""
    return oracle.score(f32(q), f32(K), f32(V), lens.cpu().numpy(), scale=scale, n_new=n_new,
                        base_mode=base_mode, base=None if base is None else base.double().cpu().numpy())


def check_scores_and_o(r, scores_gpu, o_gpu, lens, what=""):
    lens_np = lens.cpu().numpy()
    sg, og = f32(scores_gpu).astype(np.float64), f32(o_gpu)
    for b in range(len(lens_np)):
        n = int(lens_np[b])
        if n == 0:
            continue  # an empty sequence is skipped: its outputs are left as they were
        assert_close(sg[b, :, :n], r["scores"][b, :, :n], f"{what} scores[b={b}]")
        assert_close(og[b], r["o"][b], f"{what} o[b={b}]")


def check_evicted(ref_scores: np.ndarray, pos: np.ndarray, n: int, k: int, evicted_gpu, what=""):
    """One unit: the GPU's evicted slots against the oracle's choice on ITS scores, with the band rule."""
    ev_ref, _ = oracle.select_evict(ref_scores[None, None, :n], [n], [n - k], pos[None, None, :n])
    ref = set(ev_ref[0][0].tolist())
    got = set(int(x) for x in evicted_gpu)
    assert len(got) == k, f"{what}: {len(got)} distinct evicted slots, expected {k}"
    assert all(0 <= j < n for j in got), f"{what}: evicted slot out of range"
    if ref == got or k == 0:
        return 0
    tau = np.sort(ref_scores[:n])[k - 1]
    band = ATOL + RTOL * abs(tau)
    diff = ref ^ got
    for j in diff:
        assert abs(ref_scores[j] - tau) <= band, (
            f"{what}: slot {j} (score {ref_scores[j]!r}) differs from the oracle's set but is not within "
            f"{band!r} of the threshold {tau!r}")
    return len(diff)


def sub_problem(q, K, V, lens, base, units, Hkv, G):
    """Slice (b, h) units out of a batch as B' = len(units), Hkv' = 1, Hq' = G tensors."""
    qs = torch.stack([q[b, h * G:(h + 1) * G] for b, h in units])
    Ks = torch.stack([K[b, h:h + 1] for b, h in units])
    Vs = torch.stack([V[b, h:h + 1] for b, h in units])
    ls = torch.stack([lens[b] for b, h in units])
    bs = None if base is None else torch.stack([base[b, h:h + 1] for b, h in units])
    return qs, Ks, Vs, ls, bs
