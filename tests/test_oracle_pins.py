"""Pins of the CPU oracle against things it does not define itself.

Every reference value here comes from a textbook softmax attention written in this
file, finite differences of it, closed-form algebra, or brute force on tiny inputs.
A planted mistake in the oracle (dropped term, wrong sign, transposed operand,
missing count bias) must fail at least one of these.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import kvs_oracle as oc

RNG = np.random.default_rng(20240607)


# ------------------------------------------------------------------ independent reference
def ref_attention_output(q, K, V):
    """Textbook single-query softmax attention, written independently of the oracle."""
    logits = np.array([float(np.dot(q, K[i])) for i in range(K.shape[0])]) / math.sqrt(K.shape[1])
    w = np.exp(logits - np.max(logits))
    w = w / np.sum(w)
    out = np.zeros(V.shape[1])
    for i in range(K.shape[0]):
        out += w[i] * V[i]
    return out, w


def loss_linear(E, q, K, V):
    out, _ = ref_attention_output(q, K, V)
    return float(np.dot(E, out))


def fd_grad(E, q, K, V, i, h=1e-5):
    g = np.zeros(K.shape[1])
    for a in range(K.shape[1]):
        Kp, Km = K.copy(), K.copy()
        Kp[i, a] += h
        Km[i, a] -= h
        g[a] = (loss_linear(E, q, Kp, V) - loss_linear(E, q, Km, V)) / (2 * h)
    return g


def fd_hessian_block(E, q, K, V, i, j, h=1e-4):
    d = K.shape[1]
    H = np.zeros((d, d))
    for a in range(d):
        for b in range(d):
            acc = 0.0
            for sa, sb in ((1, 1), (1, -1), (-1, 1), (-1, -1)):
                Kx = K.copy()
                Kx[i, a] += sa * h
                Kx[j, b] += sb * h
                acc += sa * sb * loss_linear(E, q, Kx, V)
            H[a, b] = acc / (4 * h * h)
    return H


def tiny_problem(n=6, d=3, dv=3, seed=0):
    r = np.random.default_rng(seed)
    return (r.standard_normal(dv), r.standard_normal(d), r.standard_normal((n, d)),
            r.standard_normal((n, dv)))


# ------------------------------------------------------------------ bf16 conversion
def test_bf16_roundtrip_and_rne():
    allbits = np.arange(0x0080, 0x7F80, dtype=np.uint16)           # all positive normals
    assert np.array_equal(oc.f64_to_bf16(oc.bf16_to_f64(allbits)), allbits)
    neg = allbits | np.uint16(0x8000)
    assert np.array_equal(oc.f64_to_bf16(oc.bf16_to_f64(neg)), neg)
    # exact ties go to the even mantissa; just above a tie goes up
    lo = oc.bf16_to_f64(np.array([0x3F80, 0x3F81], dtype=np.uint16))   # 1.0, 1.0078125
    assert oc.f64_to_bf16(np.array([(lo[0] + lo[1]) / 2]))[0] == 0x3F80
    hi = oc.bf16_to_f64(np.array([0x3F82], dtype=np.uint16))
    assert oc.f64_to_bf16(np.array([(lo[1] + hi[0]) / 2]))[0] == 0x3F82
    assert oc.f64_to_bf16(np.array([(lo[0] + lo[1]) / 2 + 1e-12]))[0] == 0x3F81
    # carry into the exponent
    top = oc.bf16_to_f64(np.array([0x3FFF], dtype=np.uint16))[0]      # 1.9921875
    assert oc.f64_to_bf16(np.array([top + 0.005]))[0] == 0x4000       # -> 2.0
    # float32 semantics agree on random values
    x = RNG.standard_normal(10000) * 5
    f32 = x.astype(np.float32).astype(np.float64)                     # exact in f32 first
    u = f32.astype(np.float32).view(np.uint32)
    want = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    assert np.array_equal(oc.f64_to_bf16(f32), want)
    assert oc.f64_to_bf16(np.array([0.0, -0.0])).tolist() == [0, 0x8000]


# ------------------------------------------------------------------ Section 4.1 pins
def test_attention_matches_textbook():
    E, q, K, V = tiny_problem(7, 4, 5, 1)
    _, alpha, o = oc.attention(q, K, V)
    o_ref, a_ref = ref_attention_output(q, K, V)
    assert np.allclose(alpha, a_ref, rtol=0, atol=1e-15)
    assert np.allclose(o, o_ref, rtol=0, atol=1e-15)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_key_gradient_vs_finite_differences(seed):
    E, q, K, V = tiny_problem(6, 3, 3, seed)
    for i in range(K.shape[0]):
        g = oc.key_gradient(E, q, K, V, i)
        assert np.allclose(g, fd_grad(E, q, K, V, i), rtol=1e-6, atol=1e-9)


@pytest.mark.parametrize("seed", [0, 3])
def test_hessian_blocks_vs_finite_differences(seed):
    E, q, K, V = tiny_problem(5, 3, 3, seed)
    for m in (0, 2, 3):
        h11, h22, h12 = oc.hessian_blocks(E, q, K, V, m)
        scale = max(np.abs(h11).max(), np.abs(h22).max(), np.abs(h12).max())
        assert np.allclose(h11, fd_hessian_block(E, q, K, V, m, m), atol=2e-6 * max(scale, 1))
        assert np.allclose(h22, fd_hessian_block(E, q, K, V, m + 1, m + 1), atol=2e-6 * max(scale, 1))
        assert np.allclose(h12, fd_hessian_block(E, q, K, V, m, m + 1), atol=2e-6 * max(scale, 1))
        # symmetry of the coupling block h^{m+1,m} = h^{m,m+1} (rank one in q q^T)
        assert np.allclose(h12, fd_hessian_block(E, q, K, V, m + 1, m).T, atol=2e-6 * max(scale, 1))


def test_c_vectors_recovered_from_fd_hessian_with_unit_E():
    """With E = unit vector a, the Hessian scalar is component a of c_ij: the brute-force
    Hessian therefore pins every component and the sign of c11, c22 and c12."""
    _, q, K, V = tiny_problem(5, 2, 3, 11)
    m = 1
    _, alpha, o = ref_attention_output(q, K, V)[1], None, None
    out, w = ref_attention_output(q, K, V)
    c11, c22, c12 = oc.c_vectors(w[m], w[m + 1], V[m], V[m + 1], out)
    qq = np.outer(q, q) / K.shape[1]
    for a in range(V.shape[1]):
        E = np.zeros(V.shape[1])
        E[a] = 1.0
        for blk, cvec in (((m, m), c11), ((m + 1, m + 1), c22), ((m, m + 1), c12)):
            H = fd_hessian_block(E, q, K, V, *blk)
            coef = float(np.sum(H * qq) / np.sum(qq * qq))
            assert abs(coef - cvec[a]) < 5e-7, (blk, a, coef, cvec[a])


def test_softmax_second_derivative_identity():
    """d2 alpha_i / dz_i^2 = alpha_i(1-alpha_i)(1-2 alpha_i); the paper's diagonal coefficient
    alpha(1-2 alpha) is what multiplies (v_i - o) once the d o/dz term is included.  Check the
    resulting d s_i/d e_j of Section 4.1 by finite differences in logit space."""
    r = np.random.default_rng(5)
    z = r.standard_normal(5)
    V = r.standard_normal((5, 3))

    def s_vec(zz, i):
        a = np.exp(zz - zz.max())
        a /= a.sum()
        return a[i] * (V[i] - a @ V)

    a = np.exp(z - z.max())
    a /= a.sum()
    o = a @ V
    h = 1e-6
    for i, j in itertools.product(range(3), range(3)):
        zp, zm = z.copy(), z.copy()
        zp[j] += h
        zm[j] -= h
        fd = (s_vec(zp, i) - s_vec(zm, i)) / (2 * h)
        if i == j:
            c, _, _ = oc.c_vectors(a[i], a[i], V[i], V[i], o)
            assert np.allclose(fd, c, atol=1e-8)
        else:
            _, _, c = oc.c_vectors(a[i], a[j], V[i], V[j], o)
            assert np.allclose(fd, c, atol=1e-8)


# ------------------------------------------------------------------ Section 4.2 pins
@pytest.mark.parametrize("seed", [0, 4, 9])
def test_linear_system_and_weight_form(seed):
    E, q, K, V = tiny_problem(6, 4, 3, seed)
    m = 2
    h11, h22, h12 = oc.hessian_blocks(E, q, K, V, m)
    Mmat = h11 + 2 * h12 + h22
    Nvec = h11 @ K[m] + h12 @ (K[m] + K[m + 1]) + h22 @ K[m + 1]
    kstar = oc.projected_solution(E, q, K, V, m)
    assert np.allclose(Mmat @ kstar, Nvec, atol=1e-12)
    # minimum-norm solution equals numpy's pseudo-inverse solution
    assert np.allclose(kstar, np.linalg.pinv(Mmat) @ Nvec, atol=1e-9)
    out, w = ref_attention_output(q, K, V)
    c11, c22, c12 = oc.c_vectors(w[m], w[m + 1], V[m], V[m + 1], out)
    wm, wn = oc.exact_weights(E, c11, c22, c12)
    assert abs(wm + wn - 1.0) < 1e-12
    kw = wm * K[m] + wn * K[m + 1]
    # same component along q (the only direction the rank-one system constrains)
    assert abs(float(q @ kw) - float(q @ kstar)) < 1e-10
    assert np.allclose(Mmat @ kw, Nvec, atol=1e-12)


def test_norm_form_equals_exact_weights_when_cosines_align():
    """d_v = 1, residuals of one sign, alpha < 1/2: cos(E,c11) = cos(E,c22) = -cos(E,c12)
    holds exactly, so the gradient-free weight equals the exact one."""
    r = np.random.default_rng(3)
    n = 8
    K = r.standard_normal((n, 4)) * 0.3
    q = r.standard_normal(4)
    V = r.uniform(0.0, 0.2, size=(n, 1))
    m = 3
    V[m] = 2.0
    V[m + 1] = 3.0          # both far above o: same-sign residuals
    out, w = ref_attention_output(q, K, V)
    assert w[m] < 0.5 and w[m + 1] < 0.5 and V[m] > out and V[m + 1] > out
    c11, c22, c12 = oc.c_vectors(w[m], w[m + 1], V[m], V[m + 1], out)
    for E in (np.array([1.0]), np.array([-2.5])):
        wm, _ = oc.exact_weights(E, c11, c22, c12)
        wn = oc.norm_form_weight(np.linalg.norm(c11), np.linalg.norm(c22), np.linalg.norm(c12))
        assert abs(wm - wn) < 1e-12


def test_norm_form_weight_closed_form_and_guards():
    assert oc.norm_form_weight(3.0, 1.0, 0.5) == pytest.approx((3 - 0.5) / (3 - 1 + 1))
    assert oc.norm_form_weight(1.0, 3.0, 0.5) == pytest.approx((1 - 0.5) / 3)
    assert oc.norm_form_weight(1.0, 1.0, 1.0) == 0.5            # zero denominator
    assert oc.norm_form_weight(0.0, 0.0, 0.0) == 0.5
    assert oc.norm_form_weight(1.0, 5.0, 2.0) == 0.0            # (1-2)/(1-4+5) < 0 -> clip
    assert oc.norm_form_weight(5.0, 1.0, 2.0) == 1.0            # (5-2)/(2) > 1 -> clip
    assert oc.norm_form_weight(float("nan"), 1.0, 0.1) == 0.5


# ------------------------------------------------------------------ window statistics
def _rand_bf16(shape, r, scale=1.0):
    x = (r.standard_normal(shape) * scale).astype(np.float32)
    u = x.view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def test_window_stats_against_per_query_definitions():
    """N1, N12 and A are sums over the window queries of per-query quantities that are
    themselves pinned above (c-vectors).  Rebuild them query by query with the textbook
    attention, with the causal mask expressed by truncating the key list."""
    r = np.random.default_rng(8)
    n, d, G, W = 20, 6, 2, 3
    Kb, Vb, Qb = _rand_bf16((n, d), r), _rand_bf16((n, d), r), _rand_bf16((G, W, d), r)
    c = np.ones(n)
    Kf, Vf, Qf = oc.bf16_to_f64(Kb), oc.bf16_to_f64(Vb), oc.bf16_to_f64(Qb)
    scale = 0.37
    alpha, o, vbar = oc.window_probabilities(Kf, Vf, c, Qf, W, scale, True)
    A, N1 = oc.slot_stats(alpha, o, vbar)
    off, P = 2, 6
    N12, cosv, score = oc.pair_stats(Kf, alpha, o, vbar, A, off, P, 0)
    A_ref, N1_ref, N12_ref = np.zeros(n), np.zeros(n), np.zeros(P)
    for g in range(G):
        for i in range(W):
            vis = n - W + i + 1                                   # slots 0..n-W+i
            qeff = Qf[g, i] * scale * math.sqrt(d)                 # textbook divides by sqrt(d)
            out, w = ref_attention_output(qeff, Kf[:vis], Vf[:vis])
            assert np.allclose(alpha[g * W + i, :vis], w, atol=1e-15)
            assert np.all(alpha[g * W + i, vis:] == 0)
            A_ref[:vis] += w
            for j in range(vis):
                c11, _, _ = oc.c_vectors(w[j], w[j], Vf[j], Vf[j], out)
                N1_ref[j] += np.linalg.norm(c11)
            for p in range(P):
                j = off + 2 * p
                if j + 1 < vis:
                    _, _, c12 = oc.c_vectors(w[j], w[j + 1], Vf[j], Vf[j + 1], out)
                    N12_ref[p] += np.linalg.norm(c12)
    assert np.allclose(A, A_ref, atol=1e-14)
    assert np.allclose(N1, N1_ref, atol=1e-14)
    assert np.allclose(N12, N12_ref, atol=1e-14)
    for p in range(P):
        j = off + 2 * p
        cs = float(Kf[j] @ Kf[j + 1]) / math.sqrt(float(Kf[j] @ Kf[j]) * float(Kf[j + 1] @ Kf[j + 1]))
        assert abs(cosv[p] - cs) < 1e-14
        assert abs(score[p] - (A_ref[j] + A_ref[j + 1]) * max(0.0, 1 - cs)) < 1e-14
    _, _, score1 = oc.pair_stats(Kf, alpha, o, vbar, A, off, P, 1)
    assert np.allclose(score1, A_ref[off:off + 2 * P:2] + A_ref[off + 1:off + 2 * P:2], atol=1e-14)


def test_merged_slot_equals_its_expanded_tokens():
    """A slot with count c, value sum S and key k must behave exactly like c tokens that all
    have key k and whose values sum to S: same o, same total mass.  Pins ln(c) and S/c."""
    r = np.random.default_rng(12)
    n, d, G, W = 9, 4, 1, 2
    Kf = r.standard_normal((n, d))
    V = r.standard_normal((n + 2, d))
    Q = r.standard_normal((G, W, d))
    # expanded cache: slot 2 is three tokens with the same key
    K_exp = np.concatenate([Kf[:2], Kf[2:3], Kf[2:3], Kf[2:3], Kf[3:]], axis=0)
    a_exp, o_exp, _ = oc.window_probabilities(K_exp, V, np.ones(n + 2), Q, W, 0.5, False)
    Vsum = np.concatenate([V[:2], V[2:5].sum(0, keepdims=True), V[5:]], axis=0)
    c = np.ones(n)
    c[2] = 3
    a_m, o_m, vbar = oc.window_probabilities(Kf, Vsum, c, Q, W, 0.5, False)
    assert np.allclose(o_m, o_exp, atol=1e-14)
    assert np.allclose(a_m[:, 2], a_exp[:, 2:5].sum(1), atol=1e-14)
    assert np.allclose(a_m[:, 3:], a_exp[:, 5:], atol=1e-14)
    assert np.allclose(vbar[2], V[2:5].mean(0), atol=1e-15)


def test_causal_mask_positions():
    r = np.random.default_rng(2)
    n, d, G, W = 10, 4, 2, 4
    alpha, _, _ = oc.window_probabilities(r.standard_normal((n, d)), r.standard_normal((n, d)),
                                          np.ones(n), r.standard_normal((G, W, d)), W, 1.0, True)
    for g in range(G):
        for i in range(W):
            row = alpha[g * W + i]
            assert np.all(row[: n - W + i + 1] > 0) and np.all(row[n - W + i + 1:] == 0)
            assert abs(row.sum() - 1) < 1e-14


# ------------------------------------------------------------------ selection / schedule
def test_select_pairs_brute_force_with_ties():
    r = np.random.default_rng(4)
    for trial in range(50):
        P = int(r.integers(1, 12))
        score = r.integers(0, 4, size=P).astype(np.float64)        # many ties
        R = int(r.integers(0, P + 1))
        want = sorted(range(P), key=lambda p: (score[p], p))[:R]
        mask = oc.select_pairs(score, R)
        assert mask.sum() == R and sorted(np.nonzero(mask)[0].tolist()) == sorted(want)


def test_round_plan_closed_forms():
    # the paper's operating regime: budget 2048 + chunk 512, sink 32 -> one round of 512 merges
    plan = oc.full_plan(2560, 2048, 32, 32, 0.5)
    assert plan == [(2560, 32, (2560 - 32 - 32) // 2, 512)]
    # parity alternates, every round removes R, ends exactly on the budget
    plan = oc.full_plan(4096, 1024, 32, 32, 0.5)
    n = 4096
    for r, (nr, off, P, R) in enumerate(plan):
        assert nr == n and off == 32 + r % 2 and P == (n - off - 32) // 2
        assert R == min(n - 1024, max(1, P // 2))
        n -= R
    assert n == 1024 and len(plan) == 5
    assert len(oc.full_plan(32768, 2048, 32, 64, 0.5)) == 10
    assert len(oc.full_plan(131072, 4096, 32, 128, 0.5)) == 13
    with pytest.raises(ValueError):
        oc.full_plan(70, 10, 32, 32, 0.5)        # protected regions exceed the budget
    assert oc.full_plan(100, 100, 32, 32, 0.5) == []
    assert oc.round_plan(100, 99, 32, 32, 0.01, 0) == (32, 18, 1)     # at least one pair


# ------------------------------------------------------------------ merge + compaction
def test_apply_merge_bookkeeping():
    r = np.random.default_rng(6)
    n, d, off, P = 30, 8, 3, 10
    Kb, Vb = _rand_bf16((n, d), r, 3.0), _rand_bf16((n, d), r, 3.0)
    c = r.integers(1, 5, size=n)
    mask = np.zeros(P, dtype=np.uint8)
    mask[[0, 3, 4, 9]] = 1
    w = r.uniform(0, 1, size=P)
    Kn, Vn, cn, idx = oc.apply_merge(Kb, Vb, c, off, mask, w)
    assert Kn.shape[0] == n - 4 and cn.sum() == c.sum()
    Kf, Vf = oc.bf16_to_f64(Kb), oc.bf16_to_f64(Vb)
    # monotone, stable map; right members land on their partner
    assert np.all(np.diff(idx) >= 0) and idx[0] == 0 and idx[-1] == n - 5
    for p in range(P):
        j = off + 2 * p
        if mask[p]:
            assert idx[j] == idx[j + 1]
            want = Kf[j + 1] + w[p] * (Kf[j] - Kf[j + 1])
            got = oc.bf16_to_f64(Kn[idx[j]])
            # round to nearest: error at most half a bf16 ulp, and ulp <= |x| 2^-7
            assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8)
            vs = Vf[j] + Vf[j + 1]
            assert np.all(np.abs(oc.bf16_to_f64(Vn[idx[j]]) - vs) <= np.abs(vs) * 2.0 ** -8)
            assert cn[idx[j]] == c[j] + c[j + 1]
        else:
            assert idx[j + 1] == idx[j] + 1
            assert np.array_equal(Kn[idx[j]], Kb[j]) and np.array_equal(Kn[idx[j + 1]], Kb[j + 1])
            assert np.array_equal(Vn[idx[j]], Vb[j]) and cn[idx[j + 1]] == c[j + 1]
    # untouched prefix and suffix are bit-identical and keep their order
    assert np.array_equal(Kn[:off], Kb[:off]) and np.array_equal(Vn[-(n - off - 2 * P):], Vb[off + 2 * P:])
    # total value mass is conserved up to the bf16 rounding of the merged rows
    assert np.allclose(oc.bf16_to_f64(Vn).sum(0), Vf.sum(0), atol=4 * 2.0 ** -7 * 12)


def test_merge_unit_invariants_and_identical_keys():
    r = np.random.default_rng(7)
    n, d, G, W, sink, budget = 120, 8, 2, 4, 5, 40
    Kb, Vb, Qb = _rand_bf16((n, d), r), _rand_bf16((n, d), r), _rand_bf16((G, W, d), r)
    # plant identical neighbours: they have cosine 1 -> score 0 -> merged first, K unchanged
    for j in (sink + 2, sink + 10, sink + 20):
        Kb[j + 1] = Kb[j]
    trace = []
    Kn, Vn, cn = oc.merge_unit(Kb, Vb, np.ones(n, dtype=np.int64), Qb, budget, window=W, sink=sink,
                               trace=trace)
    assert Kn.shape[0] == budget and Vn.shape[0] == budget and cn.sum() == n
    assert np.array_equal(Kn[:sink], Kb[:sink]) and np.array_equal(Vn[:sink], Vb[:sink])
    assert np.array_equal(Kn[-W:], Kb[-W:]) and np.array_equal(cn[-W:], np.ones(W))
    st = trace[0]
    for j in (sink + 2, sink + 10, sink + 20):
        p = (j - st["off"]) // 2
        assert st["score"][p] <= 1e-12 and st["mask"][p] == 1
    for t in trace:
        assert t["mask"].sum() == t["R"]
        assert np.all((t["w"] >= 0) & (t["w"] <= 1))
    # one round by hand: merging identical keys returns that key, bit for bit
    K1, V1, c1 = oc.merge_unit(Kb, Vb, np.ones(n, dtype=np.int64), Qb, budget, window=W, sink=sink,
                               max_rounds=1)
    assert np.array_equal(K1[sink + 2], Kb[sink + 2]) and c1[sink + 2] == 2


def test_value_sum_merge_is_lossless_for_identical_keys():
    """Decode over a cache in which identical-key neighbours were merged (value sum, count 2)
    equals textbook attention over the unmerged cache."""
    r = np.random.default_rng(9)
    n, d = 16, 8
    Kb, Vb = _rand_bf16((n, d), r), _rand_bf16((n, d), r)
    Kb[5] = Kb[4]
    Kb[11] = Kb[10]
    qb = _rand_bf16((2, 3, d), r)
    Kf, Vf, qf = oc.bf16_to_f64(Kb), oc.bf16_to_f64(Vb), oc.bf16_to_f64(qb)
    keep = np.ones(n, dtype=bool)
    keep[[5, 11]] = False
    Vsum = Vf.copy()
    Vsum[4] += Vf[5]
    Vsum[10] += Vf[11]
    c = np.ones(n, dtype=np.int64)
    c[[4, 10]] = 2
    # value sums of two bf16 numbers need not be bf16; keep them exact by using float input bits
    Vsum_bits = oc.f64_to_bf16(Vsum[keep])
    exact = np.array_equal(oc.bf16_to_f64(Vsum_bits), Vsum[keep])
    out, lse = oc.decode_attention(qb, Kb[keep], Vsum_bits, c[keep])
    for g in range(2):
        for t in range(3):
            ref, w = ref_attention_output(qf[g, t], Kf, Vf)
            tol = 1e-13 if exact else 2e-2
            assert np.allclose(out[g, t], ref, atol=tol)
            e = Kf @ qf[g, t] / math.sqrt(d)
            assert abs(lse[g, t] - (np.log(np.sum(np.exp(e - e.max()))) + e.max())) < 1e-12


def test_decode_counts_one_is_textbook_attention():
    r = np.random.default_rng(10)
    n, d = 33, 16
    Kb, Vb, qb = _rand_bf16((n, d), r), _rand_bf16((n, d), r), _rand_bf16((3, 2, d), r)
    out, _ = oc.decode_attention(qb, Kb, Vb, np.ones(n, dtype=np.int64))
    for g in range(3):
        for t in range(2):
            ref, _ = ref_attention_output(oc.bf16_to_f64(qb)[g, t], oc.bf16_to_f64(Kb), oc.bf16_to_f64(Vb))
            assert np.allclose(out[g, t], ref, atol=1e-13)


def test_forced_mask_is_followed():
    r = np.random.default_rng(13)
    n, d, G, W, sink, budget = 60, 8, 1, 4, 4, 50
    Kb, Vb, Qb = _rand_bf16((n, d), r), _rand_bf16((n, d), r), _rand_bf16((G, W, d), r)
    off, P, R = oc.round_plan(n, budget, sink, W, 0.5, 0)
    forced = np.zeros(P, dtype=np.uint8)
    forced[:R] = 1
    Kn, Vn, cn = oc.merge_unit(Kb, Vb, np.ones(n, dtype=np.int64), Qb, budget, window=W, sink=sink,
                               forced_masks=[forced])
    assert np.array_equal(cn[sink:sink + R], np.full(R, 2))


def test_n1_is_a_norm_when_attention_is_peaked():
    """alpha > 1/2 makes (1 - 2 alpha) negative; N1 sums NORMS of c_jj, so it uses |1 - 2 alpha|."""
    r = np.random.default_rng(14)
    n, d = 5, 4
    Kf = r.standard_normal((n, d)) * 0.1
    Q = r.standard_normal((1, 1, d))
    Kf[1] = 6.0 * Q[0, 0] / np.linalg.norm(Q[0, 0])          # one dominant key
    V = r.standard_normal((n, d))
    alpha, o, vbar = oc.window_probabilities(Kf, V, np.ones(n), Q, 1, 1.0, False)
    assert alpha[0, 1] > 0.5
    _, N1 = oc.slot_stats(alpha, o, vbar)
    c11, _, _ = oc.c_vectors(alpha[0, 1], alpha[0, 1], V[1], V[1], o[0])
    assert N1[1] > 0 and abs(N1[1] - np.linalg.norm(c11)) < 1e-14


def test_streaming_steps_keep_the_token_and_value_books():
    """Three streaming steps (append a chunk, merge back to the budget): after every step the
    cache holds exactly `budget` slots, the counts add up to all tokens seen, the sink slots
    and the chunk's last `window` tokens are bit-identical to what was appended, the value sums
    add up to the sum of all token values (each merge adds two bf16 numbers and rounds once),
    and a step whose chunk fits the budget leaves the cache as the plain concatenation."""
    rng = np.random.default_rng(5)
    d, W, G, sink, budget, chunk = 16, 4, 2, 4, 40, 12
    bits = lambda x: oc.f64_to_bf16(np.asarray(x, dtype=np.float64))
    K = bits(rng.standard_normal((30, d))); V = bits(rng.standard_normal((30, d)))
    c = np.ones(30, dtype=np.int64)
    total_v = oc.bf16_to_f64(V).sum(0)
    seen = 30
    for step in range(3):
        cK = bits(rng.standard_normal((chunk, d))); cV = bits(rng.standard_normal((chunk, d)))
        Q = bits(rng.standard_normal((G, W, d)))
        n_before = K.shape[0]
        K2, V2, c2 = oc.append_and_merge(K, V, c, cK, cV, Q, budget, window=W, sink=sink)
        seen += chunk
        total_v = total_v + oc.bf16_to_f64(cV).sum(0)
        assert K2.shape[0] == min(budget, n_before + chunk) and int(c2.sum()) == seen
        if n_before + chunk <= budget:                     # nothing to merge yet: a plain append
            assert np.array_equal(K2, np.concatenate([K, cK])) and np.array_equal(V2, np.concatenate([V, cV]))
        assert np.array_equal(K2[:sink], K[:sink]) and np.array_equal(V2[:sink], V[:sink])
        assert np.array_equal(K2[-W:], cK[-W:]) and np.array_equal(V2[-W:], cV[-W:])
        assert np.all(c2[-W:] == 1)
        # value sums: every merged slot rounds a sum of bf16 numbers once per merge
        err = np.abs(oc.bf16_to_f64(V2).sum(0) - total_v)
        assert np.all(err <= 2.0 ** -8 * np.abs(oc.bf16_to_f64(V2)).sum(0) + 1e-12)
        K, V, c = K2, V2, c2.astype(np.int64)
    assert K.shape[0] == budget and c.max() > 1


def test_streaming_step_in_the_paper_setting_is_one_round():
    """Budget 2048 + chunk 512 with 32 sink tokens [Section 5.1]: the schedule needs one round,
    which merges exactly 512 of the candidate pairs."""
    plan = oc.full_plan(2048 + 512, 2048, 32, 64, 0.5)
    assert len(plan) == 1 and plan[0][3] == 512 and plan[0][2] >= 2 * 512


# ------------------------------------------------------------------ Eq. kstar_final inside the pass
def _bf16_exact(x):
    """Round to bf16 and return (bits, float64 values): both sides then see the same numbers."""
    bits = oc.f64_to_bf16(np.asarray(x, dtype=np.float64))
    return bits, oc.bf16_to_f64(bits)


def _fd_scalar(E, q, K, V, i, j):
    """g_ij of h^{ij} = (g_ij / d_k) q q^T, read off the finite-difference Hessian block."""
    qq = np.outer(q, q) / K.shape[1]
    H = fd_hessian_block(E, q, K, V, i, j, h=2e-4)
    return float(np.sum(H * qq) / np.sum(qq * qq))


def _aligned_tiny_cache(seed):
    """One query, d_v = 1, every value far above the attention output on one side (so all residuals
    v - o have one sign), no probability above 1/2, and candidate pairs that are far from symmetric."""
    r = np.random.default_rng(seed)
    n, d = 9, 4
    Kb, Kf = _bf16_exact(r.standard_normal((n, d)) * 0.8)
    qb, qf = _bf16_exact(r.standard_normal((1, 1, d)))
    v = r.uniform(-9.0, -7.0, size=(n, 1))                   # the protected slots pull o down
    v[1:7, 0] = [4.0, 6.0, 7.0, 5.0, 9.0, 6.5]              # the candidate slots, all above o
    Vb, Vf = _bf16_exact(v)
    return n, d, Kb, Kf, qb, qf, Vb, Vf


@pytest.mark.parametrize("seed", [21, 22, 23])
def test_round_weights_equal_exact_hessian_weights_in_the_aligned_case(seed):
    """Where Eq. cos_sign_relation_supp1 holds exactly (d_v = 1, residuals of one sign, alpha < 1/2) the
    weight that the pass applies must be the exact w_m = (g11 + g12) / gamma of
    Eq. kstar_weight_final_rewrite, with g_ij taken from a finite-difference Hessian of textbook
    attention.  Pairs are asymmetric, so a swapped pair, a shifted slot index or a constant 1/2 fails."""
    n, d, Kb, Kf, qb, qf, Vb, Vf = _aligned_tiny_cache(seed)
    sink, recent, W = 1, 2, 1
    st = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), qb, n - 1, 0, window=W, sink=sink,
                        recent=recent, scale=1.0 / math.sqrt(d), causal=True, round_frac=0.5, score_mode=0)
    assert st["off"] == 1 and st["P"] == 3
    out, alpha = ref_attention_output(qf[0, 0], Kf, Vf)
    assert alpha.max() < 0.5
    E = np.array([1.0])
    seen = []
    for p in range(st["P"]):
        m = st["off"] + 2 * p
        assert Vf[m, 0] > out[0] and Vf[m + 1, 0] > out[0]
        g11, g22, g12 = (_fd_scalar(E, qf[0, 0], Kf, Vf, m, m), _fd_scalar(E, qf[0, 0], Kf, Vf, m + 1, m + 1),
                         _fd_scalar(E, qf[0, 0], Kf, Vf, m, m + 1))
        w_exact = (g11 + g12) / (g11 + 2.0 * g12 + g22)
        assert 0.0 < w_exact < 1.0 and abs(w_exact - 0.5) > 0.03, w_exact
        assert abs(st["w"][p] - w_exact) < 2e-5, (p, st["w"][p], w_exact)
        seen.append(w_exact)
    assert max(seen) - min(seen) > 0.05                       # the pairs really differ from one another


def test_round_weights_from_per_query_norms_summed_in_the_test():
    """Several queries, causal window, merged counts: the weight of pair p must be formed from
    N1 of slot off+2p (left), N1 of slot off+2p+1 (right) and N12 of pair p, each the sum over the
    window queries of the norm of the per-query vector, all rebuilt here from textbook attention."""
    r = np.random.default_rng(31)
    n, d, dv, G, W, sink, recent = 14, 6, 5, 2, 3, 2, 3
    Kb, Kf = _bf16_exact(r.standard_normal((n, d)))
    Vb, Vf = _bf16_exact(r.standard_normal((n, dv)) * np.linspace(0.3, 3.0, n)[:, None])
    Qb, Qf = _bf16_exact(r.standard_normal((G, W, d)))
    scale = 1.0 / math.sqrt(d)
    for rnd in (0, 1):
        st = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), Qb, n - 2, rnd, window=W, sink=sink,
                            recent=recent, scale=scale, causal=True, round_frac=0.5, score_mode=0)
        off, P = st["off"], st["P"]
        assert off == sink + rnd and P == (n - off - recent) // 2
        n1 = np.zeros(n)
        n12 = np.zeros(P)
        for g in range(G):
            for i in range(W):
                vis = n - W + i + 1
                out, a = ref_attention_output(Qf[g, i], Kf[:vis], Vf[:vis])
                for j in range(vis):
                    n1[j] += a[j] * abs(1.0 - 2.0 * a[j]) * math.sqrt(float(np.sum((Vf[j] - out) ** 2)))
                for p in range(P):
                    j = off + 2 * p
                    n12[p] += a[j] * a[j + 1] * math.sqrt(float(np.sum((Vf[j] + Vf[j + 1] - 2.0 * out) ** 2)))
        ws = []
        for p in range(P):
            j = off + 2 * p
            D = n1[j] - 2.0 * n12[p] + n1[j + 1]
            assert D > 1e-3 * (n1[j] + n1[j + 1])            # well away from the guard
            want = min(1.0, max(0.0, (n1[j] - n12[p]) / D))
            assert abs(st["w"][p] - want) < 1e-12, (rnd, p, st["w"][p], want)
            ws.append(want)
        assert np.ptp(ws) > 0.02 and np.max(np.abs(np.array(ws) - 0.5)) > 0.02


def test_merge_unit_applies_the_exact_weight_to_the_left_key():
    """One round of the whole pass on the aligned tiny cache with the middle pair forced: the merged
    row must be bf16(w K_m + (1 - w) K_{m+1}) with w the finite-difference weight of the LEFT key,
    the value the sum, and everything else shifted by one slot."""
    n, d, Kb, Kf, qb, qf, Vb, Vf = _aligned_tiny_cache(22)
    sink, recent, W = 1, 2, 1
    forced = np.array([0, 1, 0], dtype=np.uint8)
    K1, V1, c1 = oc.merge_unit(Kb, Vb, np.ones(n, dtype=np.int64), qb, n - 1, window=W, sink=sink,
                               recent=recent, causal=True, round_frac=0.5, max_rounds=1,
                               forced_masks=[forced])
    m = 3
    E = np.array([1.0])
    g11, g22, g12 = (_fd_scalar(E, qf[0, 0], Kf, Vf, m, m), _fd_scalar(E, qf[0, 0], Kf, Vf, m + 1, m + 1),
                     _fd_scalar(E, qf[0, 0], Kf, Vf, m, m + 1))
    w = (g11 + g12) / (g11 + 2.0 * g12 + g22)
    want = w * Kf[m] + (1.0 - w) * Kf[m + 1]
    got = oc.bf16_to_f64(K1[m])
    assert K1.shape[0] == n - 1 and c1[m] == 2 and c1.sum() == n
    # the finite-difference weight is good to ~1e-5: allow that on top of half a bf16 ulp
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 3e-5 * np.abs(Kf[m] - Kf[m + 1]))
    # a weight of 1/2, or the weight given to the other key, would be off by many ulps on some channel
    far = np.abs(Kf[m] - Kf[m + 1]) * abs(w - 0.5)
    assert np.max(far / (np.abs(want) * 2.0 ** -8)) > 3.0
    assert np.array_equal(V1[m], oc.f64_to_bf16(Vf[m] + Vf[m + 1]))
    assert np.array_equal(K1[m + 1:], Kb[m + 2:]) and np.array_equal(K1[:m], Kb[:m])


# ------------------------------------------------------------------ Section 3.2: adjacent similarity
def test_adjacent_cosine_closed_forms():
    """Eq. cosine_raw on rows whose angles are known in closed form (all entries are small integers,
    exact in bf16): (3,4)/(4,3) -> 24/25, orthogonal -> 0, a negative multiple -> -1, a positive
    multiple -> 1, (1,1,1,1)/(1,1,0,0) -> 1/sqrt(2); the result does not depend on row scale."""
    rows = np.zeros((7, 8))
    rows[0, :2] = (3, 4)
    rows[1, :2] = (4, 3)
    rows[2, :2] = (-6, 8)            # orthogonal to (4, 3)
    rows[3, :2] = (12, -16)          # -2 x the row before
    rows[4, :2] = (48, -64)          # 4 x the row before
    rows[5, :4] = (1, 1, 1, 1)
    rows[6, :4] = (1, 1, 0, 0)
    want = np.array([24 / 25, 0.0, -1.0, 1.0, (48 - 64) / (80 * 2), 1 / math.sqrt(2)])
    got = oc.adjacent_cosine(oc.f64_to_bf16(rows))
    assert np.allclose(got, want, atol=1e-15)
    scaled = rows * np.array([1, 2, 0.5, 8, 0.25, 4, 16])[:, None]
    assert np.allclose(oc.adjacent_cosine(oc.f64_to_bf16(scaled)), want, atol=1e-15)
    assert oc.adjacent_cosine(oc.f64_to_bf16(rows[:1])).shape == (0,)
    assert oc.adjacent_cosine(oc.f64_to_bf16(np.zeros((2, 8))))[0] == 0.0      # floored denominator


def test_per_head_budgets_run_every_head_to_its_own_length():
    """Non-uniform budgets: each (sequence, KV head) ends exactly at its own budget with all of its
    tokens still counted; a head whose budget is not below its length is returned unchanged; a head
    given the sequence-wide budget gives what the per-sequence call gives."""
    r = np.random.default_rng(17)
    B, Hkv, G, W, n, d, sink = 2, 3, 2, 4, 90, 8, 4
    inputs = {"K": _rand_bf16((B, Hkv, n, d), r), "V": _rand_bf16((B, Hkv, n, d), r),
              "counts": np.ones((B, Hkv, n), dtype=np.int64), "q_win": _rand_bf16((B, Hkv * G, W, d), r),
              "seq_len": np.array([[90, 70, 90], [60, 90, 33]]), "budget": np.array([[40, 70, 25], [30, 61, 33]])}
    out = oc.merge_layer(inputs, window=W, sink=sink)
    for b in range(B):
        for h in range(Hkv):
            Kn, Vn, cn = out[(b, h)]
            n_bh, bud = inputs["seq_len"][b, h], inputs["budget"][b, h]
            assert Kn.shape[0] == min(n_bh, bud) and int(cn.sum()) == n_bh
            if bud >= n_bh:
                assert np.array_equal(Kn, inputs["K"][b, h, :n_bh])
    same = dict(inputs, seq_len=np.array([90, 60]), budget=np.array([40, 30]))
    ref = oc.merge_layer(same, window=W, sink=sink, heads=[0])
    for b in range(B):
        assert all(np.array_equal(x, y) for x, y in zip(out[(b, 0)], ref[(b, 0)]))


# ------------------------------------------------------------------ exact weights with a supplied E
def test_exact_mode_sums_and_weights_against_finite_differences():
    """weight_mode 1/2: G_ij of every candidate pair must be the sum over the window queries of the
    scalar in front of q q^T / d_k in that query's Hessian block, taken here from finite differences
    of textbook attention (causal: query i sees a truncated cache); the weight is
    (G11 + G12) / (G11 + 2 G12 + G22) [Eq. kstar_weight_final_rewrite], G11 / (G11 + G22) without
    the coupling [Eq. simplified_k], 1/2 where the denominator is not positive."""
    r = np.random.default_rng(41)
    n, d, dv, G, W, sink, recent = 11, 4, 3, 2, 2, 1, 2
    Kb, Kf = _bf16_exact(r.standard_normal((n, d)) * 0.7)
    Vb, Vf = _bf16_exact(r.standard_normal((n, dv)) * np.linspace(0.5, 2.5, n)[:, None])
    Qb, Qf = _bf16_exact(r.standard_normal((G, W, d)))
    Eb, Ef = _bf16_exact(r.standard_normal((G, W, dv)))
    kw = dict(window=W, sink=sink, recent=recent, scale=1.0 / math.sqrt(d), causal=True, round_frac=0.5, score_mode=0)
    st = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), Qb, n - 2, 0, weight_mode=1, E_bits=Eb, **kw)
    sd = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), Qb, n - 2, 0, weight_mode=2, E_bits=Eb, **kw)
    s0 = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), Qb, n - 2, 0, **kw)
    off, P = st["off"], st["P"]
    assert P == 4 and np.array_equal(st["mask"], s0["mask"]) and np.array_equal(st["score"], s0["score"])
    kinds = set()
    for p in range(P):
        m = off + 2 * p
        g11 = g22 = g12 = 0.0
        for g in range(G):
            for i in range(W):
                vis = n - W + i + 1
                g11 += _fd_scalar(Ef[g, i], Qf[g, i], Kf[:vis], Vf[:vis], m, m)
                g22 += _fd_scalar(Ef[g, i], Qf[g, i], Kf[:vis], Vf[:vis], m + 1, m + 1)
                g12 += _fd_scalar(Ef[g, i], Qf[g, i], Kf[:vis], Vf[:vis], m, m + 1)
        assert abs(st["G11"][p] - g11) < 2e-6 and abs(st["G22"][p] - g22) < 2e-6 and abs(st["G12"][p] - g12) < 2e-6
        for stx, gam, num in ((st, g11 + 2 * g12 + g22, g11 + g12), (sd, g11 + g22, g11)):
            if gam > 1e-3 * (abs(g11) + abs(g22)):
                want = min(1.0, max(0.0, num / gam))
                kinds.add("ratio" if 0.0 < want < 1.0 else "clipped")
                assert abs(stx["w"][p] - want) < 1e-4, (p, stx["w"][p], want)
            elif gam < -1e-3 * (abs(g11) + abs(g22)):
                kinds.add("guarded")
                assert stx["w"][p] == 0.5
    assert "ratio" in kinds and "guarded" in kinds
    # E -> -E flips the sign of every g: pairs with a positive denominator become guarded and the others not
    sn = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), Qb, n - 2, 0, weight_mode=1,
                        E_bits=(Eb ^ np.uint16(0x8000)), **kw)
    assert np.allclose(sn["G11"], -st["G11"]) and np.allclose(sn["G12"], -st["G12"])
    gam = st["G11"] + 2 * st["G12"] + st["G22"]
    big = np.abs(gam) > 1e-3 * (np.abs(st["G11"]) + np.abs(st["G22"]))
    assert np.all((sn["w"][big] == 0.5) == (gam[big] > 0))


def test_exact_mode_equals_norm_mode_in_the_aligned_case():
    """d_v = 1, one-sided residuals, alpha < 1/2, E > 0: the cosines of Eq. cos_sign_relation_supp1
    are exactly +1, +1, -1, so the exact weights and the gradient-free weights of Eq. kstar_final
    coincide, through the whole pass of one round."""
    n, d, Kb, Kf, qb, qf, Vb, Vf = _aligned_tiny_cache(23)
    Eb = oc.f64_to_bf16(np.full((1, 1, 1), 1.5))
    kw = dict(window=1, sink=1, recent=2, scale=1.0 / math.sqrt(d), causal=True, round_frac=0.5, score_mode=0)
    a = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), qb, n - 1, 0, **kw)
    b = oc.round_stats(Kb, Vb, np.ones(n, dtype=np.int64), qb, n - 1, 0, weight_mode=1, E_bits=Eb, **kw)
    assert np.allclose(a["w"], b["w"], atol=1e-12) and np.ptp(a["w"]) > 0.05
    K1, _, _ = oc.merge_unit(Kb, Vb, np.ones(n, dtype=np.int64), qb, n - 1, window=1, sink=1, recent=2, max_rounds=1)
    K2, _, _ = oc.merge_unit(Kb, Vb, np.ones(n, dtype=np.int64), qb, n - 1, window=1, sink=1, recent=2, max_rounds=1,
                             weight_mode=1, E_bits=Eb)
    assert np.array_equal(K1, K2)
