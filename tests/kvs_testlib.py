"""Shared helpers of the GPU parity tests: upload of generated inputs and the tolerances.

Tolerances (derived in the design notes):
  * fp32 statistics: |gpu - ref| <= 1e-5 * max(|ref|, mean|ref| over the unit);
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
