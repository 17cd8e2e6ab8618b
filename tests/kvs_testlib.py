"""Shared helpers of the GPU parity tests: upload of generated inputs and the tolerances.

Tolerances (derived in the design notes):
  * fp32 statistics A, N1, N12: plain relative error |gpu - ref| <= 1e-5 |ref| on every element
    (sums of positive terms: nothing cancels);
  * adjacent-key cosine: 1e-6 absolute; pair score = mass * (1 - cos): 1e-5 relative plus the
    cosine's absolute error times the mass (1 - cos cancels when neighbours are nearly parallel);
  * merge weight w = (N1_l - N12) / D, D = N1_l - 2 N12 + N1_r: |gpu - ref| <= 1e-5 (N1_l + N1_r +
    2 N12) / D, the first-order effect of 1e-5 relative errors in the three sums, on every pair
    above the guard on D;
  * window attention output o (an intermediate): 1e-4 of max(|ref|, mean |ref|);
  * selection mask: identical except pairs whose oracle score lies within 1e-4 (relative)
    of the selection cutoff;
  * bf16 cache rows and decode outputs: |gpu - ref| <= 2e-2, or one bf16 ulp of the
    reference element where that is larger; indices and counts bit-exact.
"""
import math

import numpy as np

from oracle import kvs_oracle as oc

STAT_RTOL = 1e-5
O_RTOL = 1e-4          # window attention output (intermediate, tensor-core accumulated)
MASK_BAND = 1e-4
BF16_ATOL = 2e-2
COS_ATOL = 1e-6
W_GUARD = 1e-6         # the guard of the weight's denominator (a reading of the paper, fixed by the oracle)


def to_dev_bf16(bits: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t) -> np.ndarray:
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def stat_close(gpu: np.ndarray, ref: np.ndarray, rtol: float = STAT_RTOL):
    """Returns (ok, worst ratio err/allowed, worst plain relative error)."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    floor = np.mean(np.abs(ref)) if ref.size else 0.0
    allowed = rtol * np.maximum(np.abs(ref), floor) + 1e-300
    err = np.abs(gpu - ref)
    ratio = float(np.max(err / allowed)) if ref.size else 0.0
    plain = float(np.max(err / np.maximum(np.abs(ref), 1e-300))) if ref.size else 0.0
    return ratio <= 1.0, ratio, plain


def rel_close(gpu: np.ndarray, ref: np.ndarray, rtol: float = STAT_RTOL, extra_abs=0.0):
    """Plain elementwise relative error.  Returns (ok, worst err / allowed, worst relative error).
    (1e-37 absolute covers values that fp32 flushes to zero.)"""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if ref.size == 0:
        return True, 0.0, 0.0
    err = np.abs(gpu - ref)
    allowed = rtol * np.abs(ref) + extra_abs + 1e-37
    return bool(np.all(err <= allowed)), float(np.max(err / allowed)), float(np.max(err / np.maximum(np.abs(ref), 1e-37)))


def check_unit_stats(got, st, label="", with_mask=True):
    """One unit's statistics from the CUDA path (`got`: arrays indexed like the oracle's, A and N1
    per slot, the others per pair) against the oracle's round_stats dictionary `st`.
    Returns {name: worst plain relative error} for reports."""
    off, P = st["off"], st["P"]
    sl = slice(off, off + 2 * P)
    worst = {}
    for name in ("A", "N1"):
        ok, ratio, plain = rel_close(got[name][sl], st[name][sl])
        worst[name] = plain
        assert ok, f"{label} {name}: worst relative error {plain:.3g} (bar {STAT_RTOL:g})"
    ok, ratio, plain = rel_close(got["N12"][:P], st["N12"][:P])
    worst["N12"] = plain
    assert ok, f"{label} N12: worst relative error {plain:.3g} (bar {STAT_RTOL:g})"
    dcos = float(np.max(np.abs(got["cos"][:P] - st["cos"][:P]))) if P else 0.0
    worst["cos_abs"] = dcos
    assert dcos <= COS_ATOL, f"{label} cos: worst absolute error {dcos:.3g}"
    mass = st["A"][off:off + 2 * P:2] + st["A"][off + 1:off + 2 * P:2]
    ok, ratio, plain = rel_close(got["score"][:P], st["score"][:P], extra_abs=COS_ATOL * mass)
    worst["score"] = plain
    assert ok, f"{label} score: err / allowed {ratio:.3g}, worst relative error {plain:.3g}"
    n1l, n1r, n12 = st["N1"][off:off + 2 * P:2], st["N1"][off + 1:off + 2 * P:2], st["N12"][:P]
    D = n1l - 2.0 * n12 + n1r
    above = D > W_GUARD * (n1l + n1r)
    bound = np.minimum(1.0, STAT_RTOL * (n1l + n1r + 2.0 * n12) / np.maximum(D, 1e-300)) + 1e-7
    dw = np.abs(got["w"][:P].astype(np.float64) - st["w"][:P])
    worst["w_over_bound"] = float(np.max((dw / bound)[above])) if np.any(above) else 0.0
    assert np.all(dw[above] <= bound[above]), f"{label} w: err / bound {worst['w_over_bound']:.3g}"
    assert np.all((got["w"][:P] >= 0) & (got["w"][:P] <= 1))
    if with_mask:
        ok, nm, nout = mask_band_ok(got["mask"][:P], st["mask"], st["score"], st["R"])
        assert ok, f"{label} mask: {nm} mismatches, {nout} outside the band"
    return worst


def mask_band_ok(mask_gpu: np.ndarray, mask_ref: np.ndarray, score_ref: np.ndarray, R: int,
                 band: float = MASK_BAND):
    """Mismatches are allowed only for pairs whose oracle score is within `band` (relative)
    of the cutoff (the R-th smallest oracle score).  Returns (ok, n_mismatch, n_outside)."""
    assert int(mask_gpu.sum()) == R, (int(mask_gpu.sum()), R)
    diff = np.nonzero(mask_gpu != mask_ref)[0]
    if diff.size == 0:
        return True, 0, 0
    cutoff = np.sort(score_ref)[R - 1]
    outside = int(np.sum(np.abs(score_ref[diff] - cutoff) > band * max(abs(cutoff), 1e-300)))
    return outside == 0, int(diff.size), outside


def bf16_close(gpu_bits: np.ndarray, ref_bits: np.ndarray, atol: float = BF16_ATOL):
    """Compare bf16 arrays.  Returns (ok, max_abs, n_one_ulp, n_worse)."""
    g = oc.bf16_to_f64(gpu_bits)
    r = oc.bf16_to_f64(ref_bits)
    err = np.abs(g - r)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(r), 2.0 ** -126))) - 7)
    allowed = np.maximum(atol, ulp)
    neq = gpu_bits != ref_bits
    worse = int(np.sum(err > allowed))
    return worse == 0, float(err.max()) if err.size else 0.0, int(np.sum(neq)), worse


def upload_layer(data):
    """numpy dict of workloads.make_layer -> dict of CUDA tensors."""
    import torch
    out = {"K": to_dev_bf16(data["K"]), "V": to_dev_bf16(data["V"]),
           "q_win": to_dev_bf16(data["q_win"]),
           "counts": torch.from_numpy(data["counts"]).cuda()}
    if data["q_new"].size:
        out["q_new"] = to_dev_bf16(data["q_new"])
    return out
