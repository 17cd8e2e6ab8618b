"""CPU float64 oracle of the KVSlimmer KV-merge pass.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It shares no code with the CUDA path and imports nothing from the package
that holds it.  It is deliberately plain and slow: numpy in float64, one
(sequence, KV head) unit at a time, no blocking or fusion, the paper's steps in the
paper's order.

What is computed (paper passages in brackets):

* attention logits, probabilities and output for the observation-window queries
  [Section 4.1, Eq. attn_def_vec], with a merged cache slot acting as one token
  whose logit carries the bias ln(count) and whose value is value_sum / count
  ["cardinality normalisation" of the value sums, Section 3.1];
* the forward-only vectors c11, c22, c12 [Section 4.2, Eqs. c11_def-c12_def], the
  key gradient [Eq. key_gradient], the Hessian blocks [Eqs. h11_mat-h22_mat], the
  linear system M k* = N and its weight-form solution [Eqs. H_gamma_rank1_rewrite,
  u_rank1_rewrite, kstar_weight_final_rewrite];
* the gradient-free merged key [Eq. kstar_final] with the norms of the c-vectors
  summed over the window queries; and, as variants of the weight only, the exact weights from a
  supplied loss gradient E [Eq. kstar_weight_final_rewrite with g_ij = E^T c_ij] and the
  diagonal-only merge that drops the coupling [Section 3.1, Eq. simplified_k];
* the value merge v* = v_m + v_{m+1} [Section 3.1] and the count bookkeeping;
* the chunk schedule "merge R adjacent pairs in parallel" [Section 3.1], repeated in
  rounds until the budget is met; the first `sink` tokens are never merged
  [Section 5.1, implementation details];
* attention over the merged cache for new queries (numerator uses value sums,
  denominator weights each slot by its count);
* the streaming step: a chunk of fresh tokens is appended and the pass brings the cache
  back to the budget [Section 3.1; Section 5.1: budget 2048, chunk 512];
* the adjacent-token cosine similarity of queries, keys or values [Section 3.2, Eq. cosine_raw].

Readings where the paper is silent are fixed here and listed in the design notes:
aligned candidate pairs with alternating parity, pair score = attention mass times
(1 - cosine), ties broken by pair index, weights clipped to [0, 1] with a guarded
denominator, |1 - 2 alpha| in the norm of c11.

Pins: tests/test_oracle_pins.py checks every function here against brute-force
finite differences of a textbook attention written in the test, closed forms,
invariants and brute-force selection on tiny inputs.  The paper prints no worked
numeric example, so agreement with "the paper's numbers" is parity unpinned; the
mathematical pins above are what the oracle stands on.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Tuple

import numpy as np

# ----------------------------------------------------------------------------- bf16


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64 (exact)."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> bf16 bit patterns, one round-to-nearest-even step straight from float64.

    Done on the float64 bit pattern so that no intermediate float32 rounding occurs.
    Inputs are assumed finite and inside the bf16 normal range (true for a KV cache).
    """
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.zeros(x.shape, dtype=np.uint16)
    nz = x != 0.0
    sign = np.signbit(x)
    m, e = np.frexp(np.abs(x[nz]))            # |x| = m * 2^e, m in [0.5, 1)
    # 8 significant bits: scale mantissa to [128, 256), round half to even
    scaled = m * 256.0
    r = np.rint(scaled)                        # numpy rint = round half to even
    carry = r >= 256.0
    r = np.where(carry, 128.0, r)
    e = e + carry.astype(e.dtype)
    exp_field = e - 1 + 127                    # value = (r/128) * 2^(e-1)
    if np.any(exp_field <= 0) or np.any(exp_field >= 255):
        # subnormal / overflow: fall back to float32 semantics (not reached by caches)
        f32 = x[nz].astype(np.float32).view(np.uint32)
        rr = f32 + np.uint32(0x7FFF) + ((f32 >> np.uint32(16)) & np.uint32(1))
        out[nz] = (rr >> np.uint32(16)).astype(np.uint16)
        return out
    bits = (exp_field.astype(np.uint32) << np.uint32(7)) | (r.astype(np.uint32) - np.uint32(128))
    bits = bits | (sign[nz].astype(np.uint32) << np.uint32(15))
    out[nz] = bits.astype(np.uint16)
    out[~nz] = np.where(sign[~nz], np.uint16(0x8000), np.uint16(0))
    return out


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bf16 value, returned as float64."""
    return bf16_to_f64(f64_to_bf16(x))


# ------------------------------------------------------------ single-query primitives
# These follow Section 4 literally for ONE query vector; the pins are stated on them.


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray,
              d_k: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """e_i = q.k_i / sqrt(d_k), alpha = softmax(e), o = sum_t alpha_t v_t  [Eq. attn_def_vec]."""
    d_k = K.shape[1] if d_k is None else d_k
    e = K @ q / math.sqrt(d_k)
    p = np.exp(e - e.max())
    alpha = p / p.sum()
    o = alpha @ V
    return e, alpha, o


def key_gradient(E: np.ndarray, q: np.ndarray, K: np.ndarray, V: np.ndarray, i: int) -> np.ndarray:
    """g_i = (1/sqrt(d_k)) alpha_i [E^T (v_i - o)] q   [Eq. key_gradient]."""
    _, alpha, o = attention(q, K, V)
    return alpha[i] * float(E @ (V[i] - o)) * q / math.sqrt(K.shape[1])


def c_vectors(alpha_m: float, alpha_n: float, v_m: np.ndarray, v_n: np.ndarray,
              o: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """c11, c22, c12 of an adjacent pair (m, n=m+1)  [Eqs. c11_def, c22_def, c12_def]."""
    c11 = alpha_m * (1.0 - 2.0 * alpha_m) * (v_m - o)
    c22 = alpha_n * (1.0 - 2.0 * alpha_n) * (v_n - o)
    c12 = -alpha_m * alpha_n * (v_m + v_n - 2.0 * o)
    return c11, c22, c12


def hessian_blocks(E: np.ndarray, q: np.ndarray, K: np.ndarray, V: np.ndarray,
                   m: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """h^{mm}, h^{m+1,m+1}, h^{m,m+1} = (1/d_k) (E^T c_ij) q q^T  [Eqs. h11_mat-h22_mat]."""
    _, alpha, o = attention(q, K, V)
    c11, c22, c12 = c_vectors(alpha[m], alpha[m + 1], V[m], V[m + 1], o)
    qq = np.outer(q, q) / K.shape[1]
    return float(E @ c11) * qq, float(E @ c22) * qq, float(E @ c12) * qq


def exact_weights(E: np.ndarray, c11: np.ndarray, c22: np.ndarray,
                  c12: np.ndarray) -> Tuple[float, float]:
    """w_m = (g11+g12)/gamma, w_{m+1} = (g12+g22)/gamma, g_ij = E^T c_ij
    [Eq. kstar_weight_final_rewrite]."""
    g11, g22, g12 = float(E @ c11), float(E @ c22), float(E @ c12)
    gamma = g11 + 2.0 * g12 + g22
    return (g11 + g12) / gamma, (g12 + g22) / gamma


def projected_solution(E: np.ndarray, q: np.ndarray, K: np.ndarray, V: np.ndarray,
                       m: int) -> np.ndarray:
    """k* = (1/gamma) P_q b, the pseudo-inverse solution of M k* = N  [Eq. kstar_proj_form]."""
    _, alpha, o = attention(q, K, V)
    c11, c22, c12 = c_vectors(alpha[m], alpha[m + 1], V[m], V[m + 1], o)
    g11, g22, g12 = float(E @ c11), float(E @ c22), float(E @ c12)
    gamma = g11 + 2.0 * g12 + g22
    b = (g11 + g12) * K[m] + (g12 + g22) * K[m + 1]
    P_q = np.outer(q, q) / float(q @ q)
    return P_q @ b / gamma


def norm_form_weight(n11: float, n22: float, n12: float) -> float:
    """Weight of k_m in the gradient-free merged key [Eq. kstar_final]:
    (|c11| - |c12|) / (|c11| - 2|c12| + |c22|).  The weight of k_{m+1} is 1 minus this.
    Guard (reading, paper silent): if the denominator is not safely positive the weight is
    1/2; the result is clipped to [0, 1] so that k* stays on the segment."""
    D = n11 - 2.0 * n12 + n22
    if not (math.isfinite(D) and D > 1e-6 * (n11 + n22)):
        return 0.5
    w = (n11 - n12) / D
    return min(1.0, max(0.0, w))


# -------------------------------------------------------------- one unit, one round


def round_plan(n: int, budget: int, sink: int, recent: int, round_frac: float,
               r: int) -> Tuple[int, int, int]:
    """Candidate layout of round r on a cache of n slots: (off, P, R).

    Candidates are the aligned pairs (off+2p, off+2p+1), p < P, between the protected
    prefix (`sink`) and the protected suffix (`recent`); the parity of `off` alternates
    with r.  R pairs are merged: the paper's "chunk_size pairs in one step" with
    chunk_size = min(n - budget, max(1, floor(round_frac * P)))."""
    off = sink + (r % 2)
    P = max(0, (n - off - recent) // 2)
    if P == 0:
        return off, 0, 0
    R = min(n - budget, max(1, int(math.floor(round_frac * P))))
    return off, P, R


def full_plan(n: int, budget: int, sink: int, recent: int, round_frac: float,
              first_round: int = 0) -> List[Tuple[int, int, int, int]]:
    """All rounds (n_r, off, P, R) until n == budget.  Raises if a round has no candidate."""
    out = []
    r = first_round
    while n > budget:
        off, P, R = round_plan(n, budget, sink, recent, round_frac, r)
        if P == 0:
            raise ValueError("budget unreachable: no candidate pair left")
        out.append((n, off, P, R))
        n -= R
        r += 1
    return out


def window_probabilities(Kf: np.ndarray, Vsum: np.ndarray, c: np.ndarray, Q: np.ndarray,
                         window: int, scale: float, causal: bool
                         ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """alpha [M, n], o [M, d_v], vbar [n, d_v] for the M = G*W window queries of one unit.

    Q is [G, W, d] (the G query heads that share this KV head, last W positions).
    Slot j has logit scale*<q, K_j> + ln c_j and value vbar_j = Vsum_j / c_j.  With
    `causal`, window query i sees slots j <= n - W + i (its own position and before)."""
    n = Kf.shape[0]
    G, W, d = Q.shape
    assert W == window
    Qm = Q.reshape(G * W, d)
    vbar = Vsum / c[:, None]
    s = scale * (Qm @ Kf.T) + np.log(c)[None, :]
    if causal:
        i = np.tile(np.arange(W), G)                       # window position of each row
        j = np.arange(n)
        s = np.where(j[None, :] > (n - W + i)[:, None], -np.inf, s)
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    alpha = p / p.sum(axis=1, keepdims=True)
    o = alpha @ vbar
    return alpha, o, vbar


def slot_stats(alpha: np.ndarray, o: np.ndarray, vbar: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """A_j = sum_q alpha_qj (accumulated attention mass) and
    N1_j = sum_q |c_jj^(q)|_2 = sum_q alpha_qj |1 - 2 alpha_qj| |vbar_j - o_q|_2
    [Eqs. c11_def, c22_def; norms summed over the window queries]."""
    A = alpha.sum(axis=0)
    n = vbar.shape[0]
    N1 = np.zeros(n)
    for j in range(n):
        dist = np.linalg.norm(vbar[j][None, :] - o, axis=1)
        N1[j] = np.sum(alpha[:, j] * np.abs(1.0 - 2.0 * alpha[:, j]) * dist)
    return A, N1


def pair_stats(Kf: np.ndarray, alpha: np.ndarray, o: np.ndarray, vbar: np.ndarray, A: np.ndarray,
               off: int, P: int, score_mode: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Per candidate pair p <-> slots (j, j+1) = (off+2p, off+2p+1):
    N12_p = sum_q |c_12^(q)|_2 = sum_q alpha_qj alpha_q,j+1 |vbar_j + vbar_j+1 - 2 o_q|_2
    [Eq. c12_def], cos_p = adjacent-key cosine similarity [Eq. cosine_raw applied to keys],
    score_p = (A_j + A_j+1) * max(0, 1 - cos_p)  (mode 0)  or  A_j + A_j+1  (mode 1)."""
    N12 = np.zeros(P)
    cosv = np.zeros(P)
    score = np.zeros(P)
    for p in range(P):
        j = off + 2 * p
        dist = np.linalg.norm((vbar[j] + vbar[j + 1])[None, :] - 2.0 * o, axis=1)
        N12[p] = np.sum(alpha[:, j] * alpha[:, j + 1] * dist)
        den = max(np.linalg.norm(Kf[j]) * np.linalg.norm(Kf[j + 1]), 1e-30)
        cosv[p] = float(Kf[j] @ Kf[j + 1]) / den
        mass = A[j] + A[j + 1]
        score[p] = mass * max(0.0, 1.0 - cosv[p]) if score_mode == 0 else mass
    return N12, cosv, score


def select_pairs(score: np.ndarray, R: int) -> np.ndarray:
    """Mask with exactly R ones: the R smallest (score, index) in lexicographic order."""
    order = np.lexsort((np.arange(score.shape[0]), score))
    mask = np.zeros(score.shape[0], dtype=np.uint8)
    mask[order[:R]] = 1
    return mask


def pair_weights(N1: np.ndarray, N12: np.ndarray, off: int, P: int) -> np.ndarray:
    """Left-key weight of every candidate pair from the summed norms [Eq. kstar_final]."""
    w = np.zeros(P)
    for p in range(P):
        j = off + 2 * p
        w[p] = norm_form_weight(float(N1[j]), float(N1[j + 1]), float(N12[p]))
    return w


def exact_pair_sums(alpha: np.ndarray, o: np.ndarray, vbar: np.ndarray, E: np.ndarray, off: int,
                    P: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Scalar sensitivities of every candidate pair with a supplied loss gradient E [M, d_v] (one row
    per window query, E_q = dL/do_q): g_ij^(q) = E_q^T c_ij^(q) [Section 4.2, text before
    Eq. h_rank1_unified], summed over the window queries (the Hessian of the summed loss is the sum
    of the per-query Hessians).  Returns G11, G22, G12 [P] and, for tolerances, Gabs [3, P]: the sums
    of the absolute values of the terms of each."""
    G11, G22, G12, Gabs = np.zeros(P), np.zeros(P), np.zeros(P), np.zeros((3, P))
    for p in range(P):
        j = off + 2 * p
        for q in range(alpha.shape[0]):
            c11, c22, c12 = c_vectors(alpha[q, j], alpha[q, j + 1], vbar[j], vbar[j + 1], o[q])
            g11, g22, g12 = float(E[q] @ c11), float(E[q] @ c22), float(E[q] @ c12)
            G11[p] += g11
            G22[p] += g22
            G12[p] += g12
            Gabs[:, p] += (abs(g11), abs(g22), abs(g12))
    return G11, G22, G12, Gabs


def exact_form_weight(g11: float, g22: float, g12: float, diagonal_only: bool = False) -> float:
    """Weight of k_m from the scalar sensitivities: (g11 + g12) / (g11 + 2 g12 + g22)
    [Eq. kstar_weight_final_rewrite]; with `diagonal_only` the coupling g12 is dropped, which is
    the diagonal-Hessian merge that the paper starts from [Section 3.1, Eq. simplified_k].
    Guard (reading, paper silent): the quadratic model has a minimum only for gamma > 0; if gamma
    is not safely positive the weight is 1/2; the result is clipped to [0, 1]."""
    if diagonal_only:
        g12 = 0.0
    gamma = g11 + 2.0 * g12 + g22
    if not (math.isfinite(gamma) and gamma > 1e-6 * (abs(g11) + abs(g22))):
        return 0.5
    return min(1.0, max(0.0, (g11 + g12) / gamma))


def apply_merge(K_bits: np.ndarray, V_bits: np.ndarray, c: np.ndarray, off: int,
                mask: np.ndarray, w: np.ndarray
                ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Merge the selected pairs and compact, keeping order.

    K* = bf16(K_{j+1} + w (K_j - K_{j+1})), Vsum* = bf16(Vsum_j + Vsum_{j+1}), c* = c_j + c_{j+1};
    the merged slot takes the left member's place, the right member is dropped.
    Returns new K bits, V bits, counts and the old-slot -> new-slot index map (a right
    member maps to its partner's new slot)."""
    n = K_bits.shape[0]
    Kf = bf16_to_f64(K_bits)
    Vf = bf16_to_f64(V_bits)
    keep = np.ones(n, dtype=bool)
    Kn = K_bits.copy()
    Vn = V_bits.copy()
    cn = c.copy()
    for p in np.nonzero(mask)[0]:
        j = off + 2 * int(p)
        Kn[j] = f64_to_bf16(Kf[j + 1] + w[p] * (Kf[j] - Kf[j + 1]))
        Vn[j] = f64_to_bf16(Vf[j] + Vf[j + 1])
        cn[j] = c[j] + c[j + 1]
        keep[j + 1] = False
    new_index = np.cumsum(keep) - 1
    new_index = new_index.astype(np.int32)
    return Kn[keep], Vn[keep], cn[keep], new_index


def round_stats(K_bits: np.ndarray, V_bits: np.ndarray, c: np.ndarray, Q_bits: np.ndarray,
                budget: int, r: int, *, window: int, sink: int, recent: int, scale: float,
                causal: bool, round_frac: float, score_mode: int, weight_mode: int = 0,
                E_bits: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Everything round r decides on the current cache of one unit (nothing is modified).

    weight_mode 0: gradient-free weights from the summed norms [Eq. kstar_final];
    1: exact weights from a supplied loss gradient E_bits (bf16 [G, W, d_v], one row per window
    query) [Eq. kstar_weight_final_rewrite]; 2: the same with the coupling term dropped
    [Eq. simplified_k].  Scores and selection do not depend on the mode."""
    n = K_bits.shape[0]
    Kf = bf16_to_f64(K_bits)
    Vs = bf16_to_f64(V_bits)
    Q = bf16_to_f64(Q_bits)
    cf = c.astype(np.float64)
    off, P, R = round_plan(n, budget, sink, recent, round_frac, r)
    if P == 0:
        raise ValueError("budget unreachable: no candidate pair left")
    alpha, o, vbar = window_probabilities(Kf, Vs, cf, Q, window, scale, causal)
    A, N1 = slot_stats(alpha, o, vbar)
    N12, cosv, score = pair_stats(Kf, alpha, o, vbar, A, off, P, score_mode)
    mask = select_pairs(score, R)
    out = {"off": off, "P": P, "R": R, "A": A, "N1": N1, "N12": N12, "cos": cosv,
           "score": score, "mask": mask, "o": o, "alpha": alpha}
    if weight_mode == 0:
        out["w"] = pair_weights(N1, N12, off, P)
    else:
        E = bf16_to_f64(E_bits).reshape(alpha.shape[0], -1)
        G11, G22, G12, Gabs = exact_pair_sums(alpha, o, vbar, E, off, P)
        out.update(G11=G11, G22=G22, G12=G12, Gabs=Gabs)
        out["w"] = np.array([exact_form_weight(G11[p], G22[p], G12[p], weight_mode == 2) for p in range(P)])
    return out


def merge_unit(K_bits: np.ndarray, V_bits: np.ndarray, c: np.ndarray, Q_bits: np.ndarray,
               budget: int, *, window: int, sink: int = 32, recent: Optional[int] = None,
               scale: Optional[float] = None, causal: bool = True, round_frac: float = 0.5,
               score_mode: int = 0, first_round: int = 0, max_rounds: Optional[int] = None,
               forced_masks: Optional[List[np.ndarray]] = None, trace: Optional[list] = None,
               weight_mode: int = 0, E_bits: Optional[np.ndarray] = None
               ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """The whole pass on one (sequence, KV head): rounds until n == budget.

    K_bits, V_bits: uint16 [n, d]; c: int [n]; Q_bits: uint16 [G, W, d].  The cache is
    stored in bf16 between rounds.  `forced_masks[i]` replaces the selection of the i-th
    executed round (used to follow another implementation's near-cutoff choices);
    `trace` collects each round's statistics."""
    recent = window if recent is None else recent
    scale = 1.0 / math.sqrt(K_bits.shape[1]) if scale is None else scale
    K_bits, V_bits, c = K_bits.copy(), V_bits.copy(), np.asarray(c).astype(np.int64).copy()
    r = first_round
    done = 0
    while K_bits.shape[0] > budget and (max_rounds is None or done < max_rounds):
        st = round_stats(K_bits, V_bits, c, Q_bits, budget, r, window=window, sink=sink,
                         recent=recent, scale=scale, causal=causal, round_frac=round_frac,
                         score_mode=score_mode, weight_mode=weight_mode, E_bits=E_bits)
        mask = st["mask"] if forced_masks is None else np.asarray(forced_masks[done], dtype=np.uint8)
        assert int(mask.sum()) == st["R"]
        if trace is not None:
            trace.append(st)
        K_bits, V_bits, c, _ = apply_merge(K_bits, V_bits, c, st["off"], mask, st["w"])
        r += 1
        done += 1
    return K_bits, V_bits, c.astype(np.int32)


def append_and_merge(K_bits: np.ndarray, V_bits: np.ndarray, c: np.ndarray,
                     chunk_K_bits: np.ndarray, chunk_V_bits: np.ndarray, Q_bits: np.ndarray,
                     budget: int, **merge_kwargs) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One streaming step on one (sequence, KV head)  [Section 3.1: the cache is compressed each
    time a chunk of new tokens has arrived; Section 5.1: budget 2048, chunk 512].

    The chunk's tokens are appended after the slots in use as fresh slots (count 1, value sum =
    value), then the merge pass brings the cache back to `budget` with `Q_bits`, the queries of
    the chunk's last W positions, as observation window.  Keyword arguments as `merge_unit`."""
    K_all = np.concatenate([K_bits, chunk_K_bits], axis=0)
    V_all = np.concatenate([V_bits, chunk_V_bits], axis=0)
    c_all = np.concatenate([np.asarray(c).astype(np.int64), np.ones(chunk_K_bits.shape[0], dtype=np.int64)])
    return merge_unit(K_all, V_all, c_all, Q_bits, budget, **merge_kwargs)


def decode_attention(q_bits: np.ndarray, K_bits: np.ndarray, V_bits: np.ndarray, c: np.ndarray,
                     scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Attention of new queries over a merged cache of one KV head.

    q_bits: uint16 [G, T, d].  out_q = sum_j exp(s_qj) Vsum_j / sum_j c_j exp(s_qj),
    s_qj = scale <q, K_j>; no causal mask.  Returns (out float64 [G, T, d_v],
    lse float64 [G, T] = ln sum_j c_j exp(s_qj))."""
    Kf = bf16_to_f64(K_bits)
    Vs = bf16_to_f64(V_bits)
    q = bf16_to_f64(q_bits)
    G, T, d = q.shape
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    s = scale * (q.reshape(G * T, d) @ Kf.T)
    mx = s.max(axis=1, keepdims=True)
    p = np.exp(s - mx)
    den = p @ c.astype(np.float64)
    out = (p @ Vs) / den[:, None]
    lse = mx[:, 0] + np.log(den)
    return out.reshape(G, T, -1), lse.reshape(G, T)


def adjacent_cosine(X_bits: np.ndarray) -> np.ndarray:
    """cos(y_t, y_t+1) = <y_t, y_t+1> / (|y_t| |y_t+1|) of consecutive rows of a bf16 matrix [n, d]
    [Section 3.2, Eq. cosine_raw]; returns float64 [n - 1] (denominator floored at 1e-30)."""
    X = bf16_to_f64(X_bits)
    out = np.zeros(max(0, X.shape[0] - 1))
    for t in range(out.shape[0]):
        den = max(np.linalg.norm(X[t]) * np.linalg.norm(X[t + 1]), 1e-30)
        out[t] = float(X[t] @ X[t + 1]) / den
    return out


def merge_layer(inputs: Dict[str, np.ndarray], *, window: int, sink: int = 32,
                recent: Optional[int] = None, causal: bool = True, round_frac: float = 0.5,
                score_mode: int = 0, heads: Optional[List[int]] = None,
                sequences: Optional[List[int]] = None) -> Dict[Tuple[int, int], tuple]:
    """All (sequence, KV head) units of one layer; returns {(b, h): (K_bits, V_bits, counts)}.
    `seq_len` and `budget` are per sequence ([B]) or, for non-uniform budgets, per (sequence,
    KV head) ([B, Hkv]): units are independent, so a head simply runs to its own budget."""
    K, V, counts, q_win = inputs["K"], inputs["V"], inputs["counts"], inputs["q_win"]
    B, Hkv = K.shape[0], K.shape[1]
    G = q_win.shape[1] // Hkv
    seq_len = np.broadcast_to(np.asarray(inputs["seq_len"]).reshape(B, -1), (B, Hkv))
    budget = np.broadcast_to(np.asarray(inputs["budget"]).reshape(B, -1), (B, Hkv))
    out = {}
    for b in (range(B) if sequences is None else sequences):
        for h in (range(Hkv) if heads is None else heads):
            n = int(seq_len[b, h])
            out[(b, h)] = merge_unit(K[b, h, :n], V[b, h, :n], counts[b, h, :n],
                                     q_win[b, h * G:(h + 1) * G], int(budget[b, h]),
                                     window=window, sink=sink, recent=recent, causal=causal,
                                     round_frac=round_frac, score_mode=score_mode)
    return out
