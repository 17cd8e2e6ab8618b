"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle."""
import math

import numpy as np
import pytest

from oracle import kvs_oracle as oc
from paper_2603_00907_b200 import workloads as wl
from tests import kvs_testlib as tl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kb():
    from paper_2603_00907_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _setup(kb, w, data, **pkw):
    import torch
    dev = tl.upload_layer(data)
    p = kb.make_params(dev["K"], dev["V"], w.n_q_heads, w.window, sink=w.sink,
                       round_frac=w.round_frac, **pkw)
    ws = torch.empty(kb.kvs_workspace_size(p, w.n_max, max(w.n_decode, 0)), dtype=torch.uint8,
                     device="cuda")
    return dev, p, ws


def _oracle_kwargs(w, **kw):
    d = dict(window=w.window, sink=w.sink, recent=w.window, scale=1.0 / math.sqrt(128),
             causal=True, round_frac=w.round_frac, score_mode=0)
    d.update(kw)
    return d


def _check_round_stats(kb, w, K, V, C, q_win, n_list, r, score_mode=0, causal=True):
    """One round of statistics on caches K,V,C (numpy, [B,Hkv,Nmax,...]) vs the oracle."""
    import torch
    data = {"K": K, "V": V, "counts": C, "q_win": q_win, "q_new": np.zeros((0,), np.uint16)}
    dev, p, ws = _setup(kb, w, data, first_round=r, score_mode=score_mode, causal=causal)
    B, Hkv, Nmax = K.shape[:3]
    G, M = w.group, w.group * w.window
    f32 = dict(dtype=torch.float32, device="cuda")
    A = torch.full((B, Hkv, Nmax), float("nan"), **f32)
    N1 = torch.full((B, Hkv, Nmax), float("nan"), **f32)
    N12, cosv, score, wgt = (torch.full((B, Hkv, Nmax // 2), float("nan"), **f32) for _ in range(4))
    mask = torch.zeros((B, Hkv, Nmax // 2), dtype=torch.uint8, device="cuda")
    o_win = torch.zeros((B, Hkv, M, 128), **f32)
    lse = torch.zeros((B, Hkv, M), **f32)
    kb.kvs_window_stats(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], n_list, list(w.budgets),
                        ws, A=A, N1=N1, N12=N12, cosv=cosv, score=score, w=wgt, mask=mask,
                        o_win=o_win, lse_win=lse)
    torch.cuda.synchronize()
    A, N1, N12, cosv, score, wgt, mask, o_win = (t.cpu().numpy() for t in
                                                 (A, N1, N12, cosv, score, wgt, mask, o_win))
    refs = {}
    report = []
    for b in range(B):
        n = n_list[b]
        if n <= w.budgets[b]:
            continue
        for h in range(Hkv):
            st = oc.round_stats(K[b, h, :n], V[b, h, :n], C[b, h, :n].astype(np.int64),
                                q_win[b, h * G:(h + 1) * G], w.budgets[b], r,
                                **_oracle_kwargs(w, score_mode=score_mode, causal=causal))
            refs[(b, h)] = st
            got = {"A": A[b, h], "N1": N1[b, h], "N12": N12[b, h], "cos": cosv[b, h], "score": score[b, h],
                   "w": wgt[b, h], "mask": mask[b, h]}
            worst = tl.check_unit_stats(got, st, label=f"unit {(b, h)} round {r}")
            # o is an intermediate formed on the tensor cores from a two-term bf16 split of the
            # probabilities: held to 1e-4 of max(|ref|, mean |ref|) (its elements cross zero)
            ok, ratio, plain = tl.stat_close(o_win[b, h], st["o"], rtol=tl.O_RTOL)
            assert ok, f"o unit {(b, h)} round {r}: err/allowed {ratio:.3g}"
            report.append((b, h, worst))
    return refs, {"mask": mask, "w": wgt, "report": report}


def _small(seed=1, **kw):
    d = dict(batch=2, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(300, 517), budgets=(100, 170))
    d.update(kw)
    return wl.small_case(seed, **d)


def test_window_stats_round0(kb):
    w = _small()
    data = wl.make_layer(w)
    _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 0)


def test_window_stats_several_query_blocks(kb):
    """group * window = 160 and 288 rows: two and three query blocks, the last one partial."""
    for seed, win, heads in ((8, 40, 8), (9, 72, 8)):
        w = _small(seed=seed, batch=1, n_q_heads=heads, n_kv_heads=2, window=win, seq_lens=(900,),
                   budgets=(300,))
        data = wl.make_layer(w)
        _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 0)
        _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 1)


def test_window_stats_many_tiles_per_cta(kb):
    """Llama head layout (8 KV heads, two sequences): few key splits, so every CTA walks several
    128-slot tiles through its TMA/MMA pipeline; the last tile of each sequence is ragged."""
    w = _small(seed=10, batch=2, n_q_heads=32, n_kv_heads=8, window=40, seq_lens=(3000, 2123),
               budgets=(1000, 700))
    data = wl.make_layer(w)
    _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 0)


def test_attention_partials_with_late_spikes(kb):
    """A few late keys aligned with one query make that row's maximum jump by far more than
    2^8 after the first tiles: the kernel must rescale its running output.  Checked on the
    attention output, the log-sum-exp and the attention mass."""
    import torch
    w = _small(seed=11, batch=1, n_q_heads=32, n_kv_heads=8, window=16, seq_lens=(4000,), budgets=(1500,))
    data = wl.make_layer(w)
    K, q = data["K"], data["q_win"]
    qf = wl.bf16_bits_to_f32(q)
    for h in range(w.n_kv_heads):
        for t, (j, row) in enumerate(((700, 3), (1900, 17), (3100, 40))):
            g, i = divmod(row, w.window)
            K[0, h, j] = wl.f32_to_bf16_bits((3.0 + t) * qf[0, h * w.group + g, i])
    dev, p, ws = _setup(kb, w, data)
    B, Hkv, Nmax, M = 1, w.n_kv_heads, w.n_max, w.group * w.window
    f32 = dict(dtype=torch.float32, device="cuda")
    A = torch.zeros((B, Hkv, Nmax), **f32)
    o_win, lse = torch.zeros((B, Hkv, M, 128), **f32), torch.zeros((B, Hkv, M), **f32)
    kb.kvs_window_stats(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [4000], [1500], ws, A=A,
                        o_win=o_win, lse_win=lse)
    torch.cuda.synchronize()
    for h in range(Hkv):
        Kf, Vf = oc.bf16_to_f64(K[0, h]), oc.bf16_to_f64(data["V"][0, h])
        Qf = oc.bf16_to_f64(q[0, h * w.group:(h + 1) * w.group])
        alpha, o, _ = oc.window_probabilities(Kf, Vf, np.ones(4000), Qf, w.window, 1 / math.sqrt(128), True)
        assert alpha.max() > 0.9                      # the spikes really dominate their rows
        ok, ratio, plain = tl.stat_close(o_win[0, h].cpu().numpy(), o, rtol=tl.O_RTOL)
        assert ok, (h, ratio, plain)
        off, P, _ = oc.round_plan(4000, 1500, w.sink, w.window, 0.5, 0)
        ok, ratio, plain = tl.rel_close(A[0, h, off:off + 2 * P].cpu().numpy(), alpha.sum(0)[off:off + 2 * P])
        assert ok, (h, ratio, plain)
        s = (Qf.reshape(M, 128) @ Kf.T) / math.sqrt(128)
        i = np.tile(np.arange(w.window), w.group)
        s = np.where(np.arange(4000)[None, :] > (4000 - w.window + i)[:, None], -np.inf, s)
        lse_ref = np.log(np.exp(s - s.max(1, keepdims=True)).sum(1)) + s.max(1)
        assert np.max(np.abs(lse[0, h].cpu().numpy() - lse_ref)) < 2e-4


def test_attention_partials_with_spikes_in_consecutive_tiles(kb):
    """Keys aligned with one query, each stronger than the one before, in six consecutive
    128-slot tiles (and in the last tile before the window): the row's stabiliser moves in tile
    after tile, so each of the kernel's two softmax teams has to pick up the value the other one
    left, rescale the shared output and carry its own part of the row sum along."""
    import torch
    w = _small(seed=12, batch=1, n_q_heads=32, n_kv_heads=8, window=16, seq_lens=(4000,), budgets=(1500,))
    data = wl.make_layer(w)
    K, q = data["K"], data["q_win"]
    qf = wl.bf16_bits_to_f32(q)
    spikes = [(128 * t + 5 + t, 0.9 + 0.65 * i) for i, t in enumerate(range(8, 14))] + [(3900, 5.2)]
    for h in range(w.n_kv_heads):
        row = 5 + 3 * h                               # a different query row per head
        g, i = divmod(row, w.window)
        for j, amp in spikes:
            K[0, h, j] = wl.f32_to_bf16_bits(amp * qf[0, h * w.group + g, i])
    dev, p, ws = _setup(kb, w, data)
    B, Hkv, Nmax, M = 1, w.n_kv_heads, w.n_max, w.group * w.window
    f32 = dict(dtype=torch.float32, device="cuda")
    A = torch.zeros((B, Hkv, Nmax), **f32)
    o_win, lse = torch.zeros((B, Hkv, M, 128), **f32), torch.zeros((B, Hkv, M), **f32)
    kb.kvs_window_stats(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [4000], [1500], ws, A=A,
                        o_win=o_win, lse_win=lse)
    torch.cuda.synchronize()
    for h in range(Hkv):
        Kf, Vf = oc.bf16_to_f64(K[0, h]), oc.bf16_to_f64(data["V"][0, h])
        Qf = oc.bf16_to_f64(q[0, h * w.group:(h + 1) * w.group])
        alpha, o, _ = oc.window_probabilities(Kf, Vf, np.ones(4000), Qf, w.window, 1 / math.sqrt(128), True)
        s = (Qf.reshape(M, 128) @ Kf.T) / math.sqrt(128)
        row = 5 + 3 * h
        growth = np.diff([s[row, j] for j, _ in spikes]) * math.log2(math.e)
        assert growth.min() > 8.0                     # every spike outgrows the stabiliser's slack of 2^8
        ok, ratio, plain = tl.stat_close(o_win[0, h].cpu().numpy(), o, rtol=tl.O_RTOL)
        assert ok, (h, ratio, plain)
        off, P, _ = oc.round_plan(4000, 1500, w.sink, w.window, 0.5, 0)
        ok, ratio, plain = tl.rel_close(A[0, h, off:off + 2 * P].cpu().numpy(), alpha.sum(0)[off:off + 2 * P])
        assert ok, (h, ratio, plain)
        i = np.tile(np.arange(w.window), w.group)
        s = np.where(np.arange(4000)[None, :] > (4000 - w.window + i)[:, None], -np.inf, s)
        lse_ref = np.log(np.exp(s - s.max(1, keepdims=True)).sum(1)) + s.max(1)
        assert np.max(np.abs(lse[0, h].cpu().numpy() - lse_ref)) < 2e-4


def test_window_stats_modes(kb):
    w = _small(seed=2, seq_lens=(260, 131), budgets=(90, 60))
    data = wl.make_layer(w)
    _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 1,
                       score_mode=1)
    _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 0,
                       causal=False)


def _oracle_round(w, K, V, C, q_win, n_list, r, w_override=None, mask_override=None):
    """Advance every unit by one oracle round.  Returns new arrays + per-unit info."""
    B, Hkv, Nmax = K.shape[:3]
    G = w.group
    Kn, Vn, Cn = np.zeros_like(K), np.zeros_like(V), np.zeros_like(C)
    idx = np.zeros((B, Hkv, Nmax), dtype=np.int32)
    n_new, info = [], {}
    for b in range(B):
        n = n_list[b]
        if n <= w.budgets[b]:
            Kn[b], Vn[b], Cn[b] = K[b], V[b], C[b]
            n_new.append(n)
            continue
        for h in range(Hkv):
            st = oc.round_stats(K[b, h, :n], V[b, h, :n], C[b, h, :n].astype(np.int64),
                                q_win[b, h * G:(h + 1) * G], w.budgets[b], r, **_oracle_kwargs(w))
            ww = st["w"] if w_override is None else w_override[b, h, :st["P"]].astype(np.float64)
            mm = st["mask"] if mask_override is None else mask_override[b, h, :st["P"]]
            k2, v2, c2, ix = oc.apply_merge(K[b, h, :n], V[b, h, :n], C[b, h, :n].astype(np.int64),
                                            st["off"], mm, ww)
            m = k2.shape[0]
            Kn[b, h, :m], Vn[b, h, :m], Cn[b, h, :m] = k2, v2, c2
            idx[b, h, :n] = ix
            info[(b, h)] = st
        n_new.append(n - info[(b, 0)]["R"])
    return Kn, Vn, Cn, idx, n_new, info


def test_compact_bit_exact_given_mask(kb):
    """Same mask and fp32 weights -> indices, counts and value sums bit-exact; keys within one
    bf16 ulp (fp32 vs float64 evaluation of the convex combination)."""
    import torch
    w = _small(seed=3)
    data = wl.make_layer(w)
    K, V, C = data["K"], data["V"], data["counts"]
    B, Hkv, Nmax = K.shape[:3]
    n_list = list(w.seq_lens)
    for r in (0, 1):
        # oracle decision, weights rounded to fp32 as the GPU stores them
        _, _, _, _, _, info = _oracle_round(w, K, V, C, data["q_win"], n_list, r)
        mask = np.zeros((B, Hkv, Nmax // 2), dtype=np.uint8)
        wgt = np.zeros((B, Hkv, Nmax // 2), dtype=np.float32)
        for (b, h), st in info.items():
            mask[b, h, :st["P"]] = st["mask"]
            wgt[b, h, :st["P"]] = st["w"].astype(np.float32)
        Kn, Vn, Cn, idx, n_new, _ = _oracle_round(w, K, V, C, data["q_win"], n_list, r,
                                                  w_override=wgt, mask_override=mask)
        dev, p, ws = _setup(kb, w, {**data, "K": K, "V": V, "counts": C}, first_round=r)
        new_index = torch.full((B, Hkv, Nmax), -1, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        n_merge = [info[(b, 0)]["R"] for b in range(B)]
        got_len = kb.kvs_compact(p, dev["K"], dev["V"], dev["counts"], torch.from_numpy(mask).cuda(),
                                 torch.from_numpy(wgt).cuda(), n_list, n_merge, ws,
                                 new_index=new_index, status_dev=status)
        torch.cuda.synchronize()
        assert status.item() == 0 and got_len == n_new
        Kg, Vg, Cg = tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy()
        ig = new_index.cpu().numpy()
        for b in range(B):
            m, n = n_new[b], n_list[b]
            assert np.array_equal(Cg[b, :, :m], Cn[b, :, :m])
            assert np.array_equal(ig[b, :, :n], idx[b, :, :n])
            assert np.array_equal(Vg[b, :, :m], Vn[b, :, :m])
            ok, mx, nulp, worse = tl.bf16_close(Kg[b, :, :m], Kn[b, :, :m], atol=0.0)
            assert ok, (mx, nulp, worse)
            assert nulp <= 0.01 * Kg[b, :, :m].size
        K, V, C, n_list = Kn, Vn, Cn, n_new


def test_compact_one_cta_per_unit_and_strided_rows(kb):
    """256 (sequence, KV head) units in one launch: every unit is compacted by a single persistent
    CTA that owns all of its tiles (no cross-CTA flags).  The cache is also given a slot stride of
    160 elements, so rows are fetched one by one.  Random valid decisions; oracle bookkeeping."""
    import torch
    w = _small(seed=13, batch=32, n_q_heads=8, n_kv_heads=8, window=8,
               seq_lens=tuple(200 + 37 * (i % 7) for i in range(32)), budgets=(64,) * 32)
    data = wl.make_layer(w)
    rng = np.random.default_rng(11)
    B, Hkv, Nmax = w.batch, w.n_kv_heads, w.n_max
    for strided in (False, True):
        K, V, C = data["K"].copy(), data["V"].copy(), data["counts"].copy()
        if strided:
            Kd = torch.zeros((B, Hkv, Nmax, 160), dtype=torch.bfloat16, device="cuda")[..., :128]
            Vd = torch.zeros((B, Hkv, Nmax, 160), dtype=torch.bfloat16, device="cuda")[..., :128]
            Kd.copy_(tl.to_dev_bf16(K)); Vd.copy_(tl.to_dev_bf16(V))
        else:
            Kd, Vd = tl.to_dev_bf16(K), tl.to_dev_bf16(V)
        Cd = torch.from_numpy(C).cuda()
        n_list = list(w.seq_lens)
        for r in (0, 1):
            off = w.sink + (r % 2)
            mask = np.zeros((B, Hkv, Nmax // 2), dtype=np.uint8)
            wgt = rng.random((B, Hkv, Nmax // 2), dtype=np.float32)
            n_merge = []
            for b in range(B):
                P = (n_list[b] - off - w.window) // 2
                R = int(rng.integers(1, P // 2))
                for h in range(Hkv):
                    mask[b, h, rng.choice(P, size=R, replace=False)] = 1
                n_merge.append(R)
            p = kb.make_params(Kd, Vd, w.n_q_heads, w.window, sink=w.sink, first_round=r)
            assert p.k_stride_t == (160 if strided else 128)
            ws = torch.empty(kb.kvs_workspace_size(p, Nmax, 0), dtype=torch.uint8, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            new_index = torch.full((B, Hkv, Nmax), -1, dtype=torch.int32, device="cuda")
            got = kb.kvs_compact(p, Kd, Vd, Cd, torch.from_numpy(mask).cuda(), torch.from_numpy(wgt).cuda(),
                                 n_list, n_merge, ws, new_index=new_index, status_dev=status)
            torch.cuda.synchronize()
            assert status.item() == 0
            Kg, Vg, Cg, ig = tl.bits_of(Kd), tl.bits_of(Vd), Cd.cpu().numpy(), new_index.cpu().numpy()
            Kn, Vn, Cn = np.zeros_like(K), np.zeros_like(V), np.zeros_like(C)
            for b in range(B):
                n, m = n_list[b], n_list[b] - n_merge[b]
                assert got[b] == m
                for h in range(Hkv):
                    P = (n - off - w.window) // 2
                    k2, v2, c2, ix = oc.apply_merge(K[b, h, :n], V[b, h, :n], C[b, h, :n].astype(np.int64), off,
                                                    mask[b, h, :P], wgt[b, h, :P].astype(np.float64))
                    Kn[b, h, :m], Vn[b, h, :m], Cn[b, h, :m] = k2, v2, c2
                    assert np.array_equal(Cg[b, h, :m], c2)
                    assert np.array_equal(ig[b, h, :n], ix)
                    assert np.array_equal(Vg[b, h, :m], v2)
                    ok, mx, nulp, worse = tl.bf16_close(Kg[b, h, :m], k2, atol=0.0)
                    assert ok, (mx, nulp, worse)
            K, V, C = Kn, Vn, Cn
            n_list = got


def full_pass_vs_oracle(kb, w, data, units=None, seq_len=None, budgets=None, exact=None):
    """The whole pass in one call; the same pass as single-round calls (it must equal their
    composition bit for bit); and, for the (sequence, KV head) `units` (all when None), the oracle
    that follows the GPU's near-cutoff choices: every deviation of the GPU's mask from the oracle's
    own must lie in the cutoff band, counts must be identical and K / value sums within the bf16
    tolerance.  `exact` = (E bits [B,Hq,W,128], weight_mode) runs the exact-weight variant.
    Returns the merged caches (numpy) and the number of band flips followed."""
    import torch
    B, Hkv, Nmax = data["K"].shape[:3]
    G = w.group
    seq_len = list(w.seq_lens) if seq_len is None else list(seq_len)
    budgets = list(w.budgets) if budgets is None else list(budgets)
    plans = [oc.full_plan(n, bud, w.sink, w.window, w.round_frac) if n > bud else []
             for n, bud in zip(seq_len, budgets)]
    rounds = max(len(pl) for pl in plans)

    if exact is None:
        merge = lambda pp, d, lens, buds, wsp, **kw: kb.kvs_merge_layer(pp, d["K"], d["V"], d["counts"], d["q_win"],
                                                                        lens, buds, wsp, **kw)
        okw = {}
    else:
        e_dev = tl.to_dev_bf16(exact[0])
        merge = lambda pp, d, lens, buds, wsp, **kw: kb.kvs_merge_layer_exact(pp, d["K"], d["V"], d["counts"], d["q_win"],
                                                                              e_dev, exact[1], lens, buds, wsp, **kw)
        okw = {"weight_mode": exact[1]}

    # (1) full pass in one call
    dev, p, ws = _setup(kb, w, data)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    new_len = merge(p, dev, seq_len, budgets, ws, status_dev=status)
    torch.cuda.synchronize()
    assert status.item() == 0 and new_len == [min(n, b) for n, b in zip(seq_len, budgets)]
    K_full, V_full, C_full = tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy()
    del dev

    # (2) the same pass as single-round calls, recording the GPU's masks
    dev2, _, ws2 = _setup(kb, w, data)
    n_list = list(seq_len)
    gpu_masks = []
    for r in range(rounds):
        pr = kb.make_params(dev2["K"], dev2["V"], w.n_q_heads, w.window, sink=w.sink,
                            round_frac=w.round_frac, first_round=r)
        mask = torch.zeros((B, Hkv, Nmax // 2), dtype=torch.uint8, device="cuda")
        kb.kvs_window_stats(pr, dev2["K"], dev2["V"], dev2["counts"], dev2["q_win"], n_list, budgets, ws2, mask=mask)
        step_budget = [plans[b][r][0] - plans[b][r][3] if r < len(plans[b]) else min(seq_len[b], budgets[b])
                       for b in range(B)]
        n_list = merge(pr, dev2, n_list, step_budget, ws2)
        gpu_masks.append(mask.cpu().numpy() if units is None else
                         {(b, h): mask[b, h].cpu().numpy() for (b, h) in units})
    torch.cuda.synchronize()
    assert n_list == new_len
    K2, V2, C2 = tl.bits_of(dev2["K"]), tl.bits_of(dev2["V"]), dev2["counts"].cpu().numpy()
    for b in range(B):
        m = new_len[b]
        assert np.array_equal(K2[b, :, :m], K_full[b, :, :m])
        assert np.array_equal(V2[b, :, :m], V_full[b, :, :m])
        assert np.array_equal(C2[b, :, :m], C_full[b, :, :m])

    # (3) oracle following the GPU's masks; every deviation from its own mask must be in the band
    flips = 0
    todo = [(b, h) for b in range(B) for h in range(Hkv)] if units is None else list(units)
    for (b, h) in todo:
        n0 = seq_len[b]
        if n0 <= budgets[b]:
            continue
        gm = (lambda r: gpu_masks[r][b, h]) if units is None else (lambda r: gpu_masks[r][(b, h)])
        forced = [gm(r)[:plans[b][r][2]] for r in range(len(plans[b]))]
        trace = []
        Ko, Vo, Co = oc.merge_unit(data["K"][b, h, :n0], data["V"][b, h, :n0],
                                   data["counts"][b, h, :n0], data["q_win"][b, h * G:(h + 1) * G],
                                   budgets[b], forced_masks=forced, trace=trace,
                                   E_bits=None if exact is None else exact[0][b, h * G:(h + 1) * G],
                                   **okw, **_oracle_kwargs(w))
        for r, st in enumerate(trace):
            if exact is not None:
                # the comparison of the merged rows presumes that no merged pair sits at the guard of
                # its denominator (there 1/2 and a clipped ratio are both within rounding)
                g12 = st["G12"] if exact[1] == 1 else 0.0
                gam = st["G11"] + 2.0 * g12 + st["G22"]
                cond = np.abs(gam) / np.maximum(st["Gabs"][0] + st["Gabs"][1] + 2.0 * st["Gabs"][2], 1e-300)
                assert cond[forced[r] != 0].min() > 5e-4, "a merged pair is ill conditioned: pick another seed"
            ok, nm, nout = tl.mask_band_ok(forced[r], st["mask"], st["score"], st["R"])
            assert ok, f"unit {(b, h)} round {r}: {nm} mask mismatches, {nout} outside the band"
            flips += nm
        m = budgets[b]
        assert np.array_equal(C_full[b, h, :m], Co)
        assert Co.sum() == n0
        okk, mxk, nulpk, _ = tl.bf16_close(K_full[b, h, :m], Ko)
        okv, mxv, nulpv, _ = tl.bf16_close(V_full[b, h, :m], Vo)
        assert okk and okv, (b, h, mxk, mxv)
    return K_full, V_full, C_full, new_len, flips


def test_merge_layer_stagewise_and_end_to_end(kb):
    """Round by round from the oracle's state (statistics, mask modulo the cutoff band, merge),
    then the whole pass in one call: it must equal the composition of single-round calls bit
    for bit, and the oracle that follows the GPU's near-cutoff choices."""
    w = _small(seed=4, seq_lens=(700, 333), budgets=(128, 64))
    data = wl.make_layer(w)
    *_, flips = full_pass_vs_oracle(kb, w, data)
    print(f"band flips followed: {flips}")


def test_more_sequences_than_one_launch_table_holds(kb):
    """150 short sequences in one call (the kernels take 128 sequences per launch, so every round
    is two launches per kernel, of 128 and of 22 sequences) against the same sequences in two
    calls of 128 and 22 (the same launch shapes, hence the same summation orders): merged caches,
    lengths and decode outputs must be identical bit for bit; the bookkeeping of a unit of the
    second table is checked too."""
    import torch
    B = 150
    w = _small(seed=31, batch=B, n_q_heads=4, n_kv_heads=2, window=8,
               seq_lens=tuple(96 + 3 * (i % 15) for i in range(B)), budgets=(64,) * B, n_decode=2)
    data = wl.make_layer(w)
    dev, p, ws = _setup(kb, w, data)
    out = torch.zeros((B, w.n_q_heads, 2, 128), dtype=torch.bfloat16, device="cuda")
    n_all = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                               list(w.budgets), ws)
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], n_all, out, ws)
    torch.cuda.synchronize()
    assert n_all == list(w.budgets)
    for lo, hi in ((0, 128), (128, B)):
        sl = slice(lo, hi)
        part = {k: np.ascontiguousarray(v[sl]) for k, v in data.items()}
        d2 = tl.upload_layer(part)
        p2 = kb.make_params(d2["K"], d2["V"], w.n_q_heads, w.window, sink=w.sink, round_frac=w.round_frac)
        out2 = torch.zeros((hi - lo, w.n_q_heads, 2, 128), dtype=torch.bfloat16, device="cuda")
        n2 = kb.kvs_merge_layer(p2, d2["K"], d2["V"], d2["counts"], d2["q_win"], list(w.seq_lens[sl]),
                                list(w.budgets[sl]), ws)
        kb.kvs_decode_attn(p2, d2["q_new"], d2["K"], d2["V"], d2["counts"], n2, out2, ws)
        torch.cuda.synchronize()
        assert n2 == n_all[sl]
        assert torch.equal(dev["K"][sl, :, :64], d2["K"][:, :, :64]) and torch.equal(dev["V"][sl, :, :64], d2["V"][:, :, :64])
        assert torch.equal(dev["counts"][sl, :, :64], d2["counts"][:, :, :64])
        assert torch.equal(out[sl], out2)
    b = 140                                               # a sequence of the second launch table
    assert int(dev["counts"][b, 0, :64].sum()) == w.seq_lens[b]
    assert torch.equal(dev["K"][b, :, :w.sink], tl.to_dev_bf16(data["K"][b:b + 1])[0, :, :w.sink])


def test_streaming_steps_match_the_oracle(kb):
    """Three streaming steps (a chunk is appended, the pass merges back to the budget) through
    kvs_append_and_merge: each step must equal, bit for bit, a plain device copy of the chunk
    followed by kvs_merge_layer, and the oracle that follows the GPU's near-cutoff choices;
    the first step's chunk still fits the budget of the second sequence (a plain append)."""
    import torch
    # (generated 240 and 140 slots long so that there is room behind the 200 and 100 slots in use)
    w = _small(seed=21, batch=2, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(240, 140), budgets=(200, 140))
    B, Hkv, G, W, chunk = w.batch, w.n_kv_heads, w.group, w.window, 36
    base = wl.make_layer(w)
    Nmax = base["K"].shape[2]
    cur0 = [200, 100]
    assert Nmax >= max(cur0) + chunk
    rng = np.random.default_rng(77)
    bits = lambda shape: wl.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    dev, p, ws = _setup(kb, w, base)        # streamed through the new entry point
    dev2, _, ws2 = _setup(kb, w, base)      # the same steps from existing calls, recording masks
    cur = list(cur0)
    ora = {(b, h): (base["K"][b, h, :cur[b]].copy(), base["V"][b, h, :cur[b]].copy(),
                    base["counts"][b, h, :cur[b]].astype(np.int64)) for b in range(B) for h in range(Hkv)}
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flips = 0
    for step in range(3):
        cK, cV = bits((B, Hkv, chunk, 128)), bits((B, Hkv, chunk, 128))
        qw = bits((B, w.n_q_heads, W, 128))
        dcK, dcV, dq = tl.to_dev_bf16(cK), tl.to_dev_bf16(cV), tl.to_dev_bf16(qw)
        new_len = kb.kvs_append_and_merge(p, dev["K"], dev["V"], dev["counts"], dcK, dcV, dq, cur,
                                          list(w.budgets), ws, status_dev=status)
        # the same step from a device copy + the single-round calls
        n_list = [c + chunk for c in cur]
        for b in range(B):
            dev2["K"][b, :, cur[b]:cur[b] + chunk] = dcK[b]
            dev2["V"][b, :, cur[b]:cur[b] + chunk] = dcV[b]
            dev2["counts"][b, :, cur[b]:cur[b] + chunk] = 1
        plans = [oc.full_plan(n, bud, w.sink, W, w.round_frac) if n > bud else [] for n, bud in zip(n_list, w.budgets)]
        gpu_masks = []
        for r in range(max(len(pl) for pl in plans)):
            pr = kb.make_params(dev2["K"], dev2["V"], w.n_q_heads, W, sink=w.sink, round_frac=w.round_frac,
                                first_round=r)
            mask = torch.zeros((B, Hkv, Nmax // 2), dtype=torch.uint8, device="cuda")
            kb.kvs_window_stats(pr, dev2["K"], dev2["V"], dev2["counts"], dq, n_list, list(w.budgets), ws2, mask=mask)
            step_budget = [plans[b][r][0] - plans[b][r][3] if r < len(plans[b]) else min(n_list[b], w.budgets[b])
                           for b in range(B)]
            n_list = kb.kvs_merge_layer(pr, dev2["K"], dev2["V"], dev2["counts"], dq, n_list, step_budget, ws2)
            gpu_masks.append(mask.cpu().numpy())
        torch.cuda.synchronize()
        assert status.item() == 0
        assert new_len == n_list == [min(c + chunk, bud) for c, bud in zip(cur, w.budgets)]
        Kg, Vg, Cg = tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy()
        for b in range(B):
            m = new_len[b]
            assert np.array_equal(Kg[b, :, :m], tl.bits_of(dev2["K"])[b, :, :m])
            assert np.array_equal(Vg[b, :, :m], tl.bits_of(dev2["V"])[b, :, :m])
            assert np.array_equal(Cg[b, :, :m], dev2["counts"].cpu().numpy()[b, :, :m])
            for h in range(Hkv):
                Ko, Vo, Co = ora[(b, h)]
                forced = [gpu_masks[r][b, h, :plans[b][r][2]] for r in range(len(plans[b]))]
                trace = []
                Ko, Vo, Co = oc.append_and_merge(Ko, Vo, Co, cK[b, h], cV[b, h], qw[b, h * G:(h + 1) * G],
                                                 w.budgets[b], forced_masks=forced, trace=trace,
                                                 **_oracle_kwargs(w))
                for r, st in enumerate(trace):
                    ok, nm, nout = tl.mask_band_ok(forced[r], st["mask"], st["score"], st["R"])
                    assert ok, f"step {step} unit {(b, h)} round {r}: {nm} mismatches, {nout} outside the band"
                    flips += nm
                assert np.array_equal(Cg[b, h, :m], Co) and Co.sum() == cur0[b] + (step + 1) * chunk
                okk, mxk, _, _ = tl.bf16_close(Kg[b, h, :m], Ko)
                okv, mxv, _, _ = tl.bf16_close(Vg[b, h, :m], Vo)
                assert okk and okv, (step, b, h, mxk, mxv)
                # the next step starts from the GPU's state (so that rounding flips do not add up)
                ora[(b, h)] = (Kg[b, h, :m].copy(), Vg[b, h, :m].copy(), Cg[b, h, :m].astype(np.int64))
        cur = new_len
    print(f"band flips followed: {flips}")


def test_streaming_edge_cases(kb):
    """An empty chunk is exactly kvs_merge_layer; a chunk into an empty cache that fits the budget
    is a plain copy with counts 1; a chunk several times the budget takes several rounds and
    equals kvs_merge_layer on the concatenation, bit for bit."""
    import torch
    w = _small(seed=22, batch=2, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(400, 260), budgets=(90, 70))
    B, Hkv = w.batch, w.n_kv_heads
    data = wl.make_layer(w)
    # (1) empty chunk
    dev, p, ws = _setup(kb, w, data)
    dev2, _, ws2 = _setup(kb, w, data)
    empty = torch.zeros((B, Hkv, 0, 128), dtype=torch.bfloat16, device="cuda")
    n1 = kb.kvs_append_and_merge(p, dev["K"], dev["V"], dev["counts"], empty, empty, dev["q_win"],
                                 list(w.seq_lens), list(w.budgets), ws)
    n2 = kb.kvs_merge_layer(p, dev2["K"], dev2["V"], dev2["counts"], dev2["q_win"], list(w.seq_lens),
                            list(w.budgets), ws2)
    torch.cuda.synchronize()
    assert n1 == n2 == list(w.budgets)
    for b in range(B):
        m = n1[b]
        assert torch.equal(dev["K"][b, :, :m], dev2["K"][b, :, :m]) and torch.equal(dev["V"][b, :, :m], dev2["V"][b, :, :m])
        assert torch.equal(dev["counts"][b, :, :m], dev2["counts"][b, :, :m])
    # (2) a chunk into an empty cache, below the budget: a copy
    dev, p, ws = _setup(kb, w, data)
    chunk = 60
    cK = dev2["K"][:, :, :chunk].contiguous() * 0 + 1.5          # any bf16 payload
    cV = tl.to_dev_bf16(data["V"][:, :, 100:100 + chunk].copy())
    dev["counts"].fill_(7)
    n3 = kb.kvs_append_and_merge(p, dev["K"], dev["V"], dev["counts"], cK, cV, dev["q_win"], [0, 0],
                                 list(w.budgets), ws)
    torch.cuda.synchronize()
    assert n3 == [60, 60]
    assert torch.equal(dev["K"][:, :, :chunk], cK) and torch.equal(dev["V"][:, :, :chunk], cV)
    assert torch.all(dev["counts"][:, :, :chunk] == 1) and torch.all(dev["counts"][:, :, chunk:] == 7)
    # (3) a large chunk behind a short cache: several rounds, equal to the pass on the concatenation
    dev, p, ws = _setup(kb, w, data)
    dev2, _, ws2 = _setup(kb, w, data)
    cur, chunk = [100, 40], 220
    cK = tl.to_dev_bf16(np.ascontiguousarray(data["K"][:, :, 30:30 + chunk]))
    cV = tl.to_dev_bf16(np.ascontiguousarray(data["V"][:, :, 30:30 + chunk]))
    for b in range(B):
        dev2["K"][b, :, cur[b]:cur[b] + chunk] = cK[b]
        dev2["V"][b, :, cur[b]:cur[b] + chunk] = cV[b]
        dev2["counts"][b, :, cur[b]:cur[b] + chunk] = 1
    n4 = kb.kvs_append_and_merge(p, dev["K"], dev["V"], dev["counts"], cK, cV, dev["q_win"], cur,
                                 list(w.budgets), ws)
    n5 = kb.kvs_merge_layer(p, dev2["K"], dev2["V"], dev2["counts"], dev2["q_win"], [c + chunk for c in cur],
                            list(w.budgets), ws2)
    torch.cuda.synchronize()
    assert n4 == n5 == list(w.budgets)
    assert len(oc.full_plan(cur[0] + chunk, w.budgets[0], w.sink, w.window, w.round_frac)) >= 3
    for b in range(B):
        m = n4[b]
        assert torch.equal(dev["K"][b, :, :m], dev2["K"][b, :, :m]) and torch.equal(dev["V"][b, :, :m], dev2["V"][b, :, :m])
        assert torch.equal(dev["counts"][b, :, :m], dev2["counts"][b, :, :m])
        assert int(dev["counts"][b, 0, :m].sum()) == cur[b] + chunk
    # (4) no room behind the slots in use: rejected on the host, nothing is touched
    before = dev["K"].clone()
    with pytest.raises(kb.KvsError):
        kb.kvs_append_and_merge(p, dev["K"], dev["V"], dev["counts"], cK, cV, dev["q_win"],
                                [w.n_max - 10, 0], list(w.budgets), ws)
    torch.cuda.synchronize()
    assert torch.equal(before, dev["K"])


def test_decode_matches_oracle_and_is_lossless_on_identical_keys(kb):
    import torch
    w = _small(seed=5, seq_lens=(400, 257), budgets=(90, 60), n_decode=5)
    data = wl.make_layer(w)
    # plant identical neighbours so that round 0 merges them first
    for b in range(w.batch):
        for j in (40, 60, 100):
            data["K"][b, :, j + 1] = data["K"][b, :, j]
    dev, p, ws = _setup(kb, w, data)
    B, Hq, T = w.batch, w.n_q_heads, w.n_decode
    G, Hkv = w.group, w.n_kv_heads
    out0 = torch.zeros((B, Hq, T, 128), dtype=torch.bfloat16, device="cuda")
    lse0 = torch.zeros((B, Hq, T), dtype=torch.float32, device="cuda")
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], list(w.seq_lens), out0, ws,
                       lse=lse0)
    torch.cuda.synchronize()
    o0 = tl.bits_of(out0)
    for b in range(B):
        n = w.seq_lens[b]
        for h in range(Hkv):
            ref, lse_ref = oc.decode_attention(data["q_new"][b, h * G:(h + 1) * G], data["K"][b, h, :n],
                                               data["V"][b, h, :n], data["counts"][b, h, :n])
            ok, mx, _, _ = tl.bf16_close(o0[b, h * G:(h + 1) * G], oc.f64_to_bf16(ref))
            assert ok, mx
            assert np.max(np.abs(lse0[b, h * G:(h + 1) * G].cpu().numpy() - lse_ref)) < 1e-4
    # merge to the budget, decode again, compare with the oracle's merged cache
    new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                                 list(w.budgets), ws)
    out1 = torch.zeros_like(out0)
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], new_len, out1, ws)
    torch.cuda.synchronize()
    Kg, Vg, Cg = tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy()
    o1 = tl.bits_of(out1)
    for b in range(B):
        m = new_len[b]
        for h in range(Hkv):
            ref, _ = oc.decode_attention(data["q_new"][b, h * G:(h + 1) * G], Kg[b, h, :m], Vg[b, h, :m],
                                         Cg[b, h, :m])
            ok, mx, _, _ = tl.bf16_close(o1[b, h * G:(h + 1) * G], oc.f64_to_bf16(ref))
            assert ok, mx


def test_decode_many_rows_and_tiles(kb):
    """group * n_new = 192 query rows (two blocks) over caches of several tiles, merged counts."""
    import torch
    w = _small(seed=12, batch=2, n_q_heads=16, n_kv_heads=4, window=8, seq_lens=(1500, 777),
               budgets=(1500, 777), n_decode=48)
    data = wl.make_layer(w)
    rng = np.random.default_rng(5)
    data["counts"][:] = rng.integers(1, 6, size=data["counts"].shape)          # as if merged before
    dev, p, ws = _setup(kb, w, data)
    B, Hq, T, G, Hkv = w.batch, w.n_q_heads, w.n_decode, w.group, w.n_kv_heads
    out = torch.zeros((B, Hq, T, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((B, Hq, T), dtype=torch.float32, device="cuda")
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], list(w.seq_lens), out, ws, lse=lse)
    torch.cuda.synchronize()
    og = tl.bits_of(out)
    for b in range(B):
        n = w.seq_lens[b]
        for h in range(Hkv):
            ref, lse_ref = oc.decode_attention(data["q_new"][b, h * G:(h + 1) * G], data["K"][b, h, :n],
                                               data["V"][b, h, :n], data["counts"][b, h, :n])
            ok, mx, _, _ = tl.bf16_close(og[b, h * G:(h + 1) * G], oc.f64_to_bf16(ref))
            assert ok, mx
            assert np.max(np.abs(lse[b, h * G:(h + 1) * G].cpu().numpy() - lse_ref)) < 1e-4


def test_identical_key_merge_is_lossless_on_gpu(kb):
    """One round that merges only planted identical-key pairs leaves decode unchanged."""
    import torch
    w = _small(seed=6, batch=1, seq_lens=(200,), budgets=(197,), n_decode=4)
    data = wl.make_layer(w)
    for j in (50, 80, 120):          # even offsets from sink=32 -> aligned candidate pairs
        data["K"][0, :, j + 1] = data["K"][0, :, j]
    dev, p, ws = _setup(kb, w, data)
    out0 = torch.zeros((1, w.n_q_heads, 4, 128), dtype=torch.bfloat16, device="cuda")
    lse0 = torch.zeros((1, w.n_q_heads, 4), dtype=torch.float32, device="cuda")
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], [200], out0, ws, lse=lse0)
    K_before = tl.bits_of(dev["K"]).copy()
    new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [200], [197], ws)
    out1, lse1 = torch.zeros_like(out0), torch.zeros_like(lse0)
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], new_len, out1, ws, lse=lse1)
    torch.cuda.synchronize()
    assert new_len == [197]
    Kg, Cg = tl.bits_of(dev["K"]), dev["counts"].cpu().numpy()
    assert np.array_equal(Cg[0, :, 50], np.full(w.n_kv_heads, 2))
    assert np.array_equal(Kg[0, :, 50], K_before[0, :, 50])                 # K* == K exactly
    assert np.array_equal(Kg[0, :, 51], K_before[0, :, 52])                 # shifted by one
    assert Cg[0, :, :197].sum() == 200 * w.n_kv_heads
    assert torch.max(torch.abs(lse1 - lse0)).item() < 1e-5
    assert torch.max(torch.abs(out1.float() - out0.float())).item() <= 2e-2


def test_noop_and_error_paths_on_device(kb):
    import torch
    w = _small(seed=7, batch=1, seq_lens=(150,), budgets=(150,))
    data = wl.make_layer(w)
    dev, p, ws = _setup(kb, w, data)
    before = tl.bits_of(dev["K"]).copy()
    assert kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [150], [150], ws) == [150]
    assert kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [100], [150], ws) == [100]
    torch.cuda.synchronize()
    assert np.array_equal(tl.bits_of(dev["K"]), before)
    with pytest.raises(kb.KvsError) as e:      # sink + recent = 40 > budget 20
        kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [150], [20], ws)
    assert e.value.code == 4
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [150], [100], ws[:1024])
    assert e.value.code == 3
    torch.cuda.synchronize()
    assert np.array_equal(tl.bits_of(dev["K"]), before)


def test_window_stats_config_layouts(kb):
    """The head layouts of the other benchmark configurations at reduced length: Qwen (7 query
    heads per KV head, 224 window rows: a partial second query block), the 70B layout (8 x 128 =
    1024 rows: eight query blocks), and a ragged batch of eight sequences."""
    for seed, kw in ((14, dict(batch=1, n_q_heads=14, n_kv_heads=2, window=32, seq_lens=(1100,), budgets=(400,))),
                     (15, dict(batch=1, n_q_heads=8, n_kv_heads=1, window=128, seq_lens=(1500,), budgets=(600,))),
                     (16, dict(batch=8, n_q_heads=8, n_kv_heads=2, window=16,
                               seq_lens=(300, 1201, 517, 64, 900, 433, 1000, 777),
                               budgets=(37, 150, 64, 64, 112, 54, 125, 97)))):
        w = _small(seed=seed, **kw)
        data = wl.make_layer(w)
        for r in (0, 1):
            _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), r)


def test_merged_counts_statistics(kb):
    """Statistics on a cache that already holds merged slots (counts > 1 carry the logit bias ln c
    and divide the value sums)."""
    w = _small(seed=17, batch=1, n_q_heads=8, n_kv_heads=2, window=16, seq_lens=(1300,), budgets=(300,))
    data = wl.make_layer(w)
    rng = np.random.default_rng(3)
    data["counts"][:] = rng.integers(1, 5, size=data["counts"].shape)
    _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 0)
    _check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], list(w.seq_lens), 1)


def test_adjacent_cosine_of_queries_keys_and_values(kb):
    """kvs_adjacent_cosine on the keys, values and (decode) queries of a ragged batch against the
    oracle, on a strided view too; entries at and behind seq_len - 1 stay untouched.  The synthetic
    keys are an AR(1) drift (homogeneous neighbours), values and queries are i.i.d."""
    import torch
    w = _small(seed=51, batch=3, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(700, 1, 333), budgets=(700, 1, 333),
               n_decode=40)
    data = wl.make_layer(w)
    dev = tl.upload_layer(data)
    B, Hkv, Nmax = w.batch, w.n_kv_heads, w.n_max
    means = {}
    for name, x, lens in (("K", dev["K"], list(w.seq_lens)), ("V", dev["V"], list(w.seq_lens)),
                          ("Q", dev["q_new"], [40, 40, 40])):
        out = torch.full(x.shape[:3], -7.0, dtype=torch.float32, device="cuda")
        kb.kvs_adjacent_cosine(x, lens, out)
        torch.cuda.synchronize()
        g = out.cpu().numpy()
        xb = tl.bits_of(x)
        acc = []
        for b in range(B):
            for h in range(x.shape[1]):
                ref = oc.adjacent_cosine(xb[b, h, :lens[b]])
                assert np.max(np.abs(g[b, h, :len(ref)] - ref), initial=0.0) < 1e-6
                assert np.all(g[b, h, len(ref):] == -7.0)
                acc.append(ref)
        means[name] = float(np.mean(np.concatenate(acc)))
    assert means["K"] > 0.8 and abs(means["V"]) < 0.05 and abs(means["Q"]) < 0.1
    # a strided view (row stride 160 elements)
    xs = torch.zeros((B, Hkv, Nmax, 160), dtype=torch.bfloat16, device="cuda")[..., :128]
    xs.copy_(dev["K"])
    out = torch.zeros((B, Hkv, Nmax), dtype=torch.float32, device="cuda")
    kb.kvs_adjacent_cosine(xs, list(w.seq_lens), out)
    torch.cuda.synchronize()
    ref = oc.adjacent_cosine(data["K"][2, 1, :333])
    assert np.max(np.abs(out[2, 1, :332].cpu().numpy() - ref)) < 1e-6


def test_per_head_budgets(kb):
    """kvs_merge_layer_per_head / kvs_decode_attn_per_head: every (sequence, KV head) runs to its own
    budget.  The same memory viewed as a batch of one-head sequences goes through the ordinary entry
    points against the oracle (band flips followed); the per-head entry points must then give those
    results bit for bit on the original layout."""
    import torch
    w = _small(seed=61, batch=2, n_q_heads=12, n_kv_heads=3, window=8, seq_lens=(600, 410), budgets=(1, 1), n_decode=2)
    data = wl.make_layer(w)
    B, Hkv, G, Nmax = w.batch, w.n_kv_heads, w.group, w.n_max
    seq_len = [600, 600, 600, 410, 410, 410]
    budget = [90, 600, 300, 64, 200, 51]
    # (1) as a batch of B * Hkv one-head sequences through the ordinary calls, against the oracle
    wu = w.scaled(batch=B * Hkv, n_q_heads=G, n_kv_heads=1, seq_lens=tuple(seq_len), budgets=tuple(budget))
    du = {"K": data["K"].reshape(B * Hkv, 1, Nmax, 128), "V": data["V"].reshape(B * Hkv, 1, Nmax, 128),
          "counts": data["counts"].reshape(B * Hkv, 1, Nmax), "q_win": data["q_win"].reshape(B * Hkv, G, w.window, 128),
          "q_new": data["q_new"].reshape(B * Hkv, G, 2, 128)}
    K_ref, V_ref, C_ref, len_ref, flips = full_pass_vs_oracle(kb, wu, du)
    assert len_ref == [min(n, b) for n, b in zip(seq_len, budget)]
    # (2) the per-head entry points on the original [B, Hkv, ...] layout
    dev = tl.upload_layer(data)
    p = kb.make_params(dev["K"], dev["V"], w.n_q_heads, w.window, sink=w.sink, round_frac=w.round_frac)
    ws = torch.empty(kb.kvs_workspace_size_per_head(p, Nmax, 2), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    new_len = kb.kvs_merge_layer_per_head(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], seq_len, budget, ws,
                                          status_dev=status)
    out = torch.zeros((B, w.n_q_heads, 2, 128), dtype=torch.bfloat16, device="cuda")
    kb.kvs_decode_attn_per_head(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], new_len, out, ws)
    torch.cuda.synchronize()
    assert status.item() == 0 and new_len == len_ref
    Kg, Vg, Cg, og = tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy(), tl.bits_of(out)
    for b in range(B):
        for h in range(Hkv):
            u, m = b * Hkv + h, new_len[b * Hkv + h]
            assert np.array_equal(Kg[b, h, :m], K_ref[u, 0, :m]) and np.array_equal(Vg[b, h, :m], V_ref[u, 0, :m])
            assert np.array_equal(Cg[b, h, :m], C_ref[u, 0, :m]) and int(Cg[b, h, :m].sum()) == seq_len[u]
            ref, _ = oc.decode_attention(data["q_new"][b, h * G:(h + 1) * G], Kg[b, h, :m], Vg[b, h, :m], Cg[b, h, :m])
            ok, mx, _, _ = tl.bf16_close(og[b, h * G:(h + 1) * G], oc.f64_to_bf16(ref))
            assert ok, ((b, h), mx)
    # a layout whose heads do not tile the sequence stride is refused
    Kbad = torch.zeros((B, Hkv + 1, Nmax, 128), dtype=torch.bfloat16, device="cuda")[:, :Hkv]
    pbad = kb.make_params(Kbad, Kbad, w.n_q_heads, w.window, sink=w.sink)
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_merge_layer_per_head(pbad, Kbad, Kbad, dev["counts"], dev["q_win"], seq_len, budget, ws)
    assert e.value.code == 2


def test_exact_weights_with_a_supplied_gradient(kb):
    """kvs_window_stats_exact / kvs_merge_layer_exact: the signed sums G_ij = sum_q E_q^T c_ij and the
    weights of both exact modes against the oracle (errors measured against the sum of the absolute
    terms, since the signed sums cancel), merged counts in the statistics, then the whole pass of a
    small cache with exact weights against the oracle."""
    import torch
    w = _small(seed=71, batch=2, n_q_heads=8, n_kv_heads=2, window=40, seq_lens=(900, 517), budgets=(300, 170))
    data = wl.make_layer(w)
    rng = np.random.default_rng(71)
    data["counts"][:] = rng.integers(1, 4, size=data["counts"].shape)
    E = wl.f32_to_bf16_bits(rng.standard_normal(data["q_win"].shape).astype(np.float32))
    dev, p, ws = _setup(kb, w, data)
    e_dev = tl.to_dev_bf16(E)
    B, Hkv, Nmax, G = w.batch, w.n_kv_heads, w.n_max, w.group
    f32 = dict(dtype=torch.float32, device="cuda")
    for r in (0, 1):
        pr = kb.make_params(dev["K"], dev["V"], w.n_q_heads, w.window, sink=w.sink, first_round=r)
        for mode in (1, 2):
            A, gs = torch.zeros((B, Hkv, Nmax), **f32), torch.zeros((B, Hkv, Nmax), **f32)
            gp, wg, sc = (torch.zeros((B, Hkv, Nmax // 2), **f32) for _ in range(3))
            mask = torch.zeros((B, Hkv, Nmax // 2), dtype=torch.uint8, device="cuda")
            kb.kvs_window_stats_exact(pr, dev["K"], dev["V"], dev["counts"], dev["q_win"], e_dev, mode,
                                      list(w.seq_lens), list(w.budgets), ws, A=A, g_self=gs, g_pair=gp, score=sc,
                                      w=wg, mask=mask)
            torch.cuda.synchronize()
            n_ratio = 0
            for b in range(B):
                n = w.seq_lens[b]
                for h in range(Hkv):
                    st = oc.round_stats(data["K"][b, h, :n], data["V"][b, h, :n], data["counts"][b, h, :n].astype(np.int64),
                                        data["q_win"][b, h * G:(h + 1) * G], w.budgets[b], r, weight_mode=mode,
                                        E_bits=E[b, h * G:(h + 1) * G], **_oracle_kwargs(w))
                    off, P = st["off"], st["P"]
                    g11, g22 = gs[b, h, off:off + 2 * P:2].cpu().numpy(), gs[b, h, off + 1:off + 2 * P:2].cpu().numpy()
                    g12 = gp[b, h, :P].cpu().numpy()
                    ab = st["Gabs"]
                    assert np.all(np.abs(g11 - st["G11"]) <= tl.STAT_RTOL * ab[0] + 1e-37)
                    assert np.all(np.abs(g22 - st["G22"]) <= tl.STAT_RTOL * ab[1] + 1e-37)
                    assert np.all(np.abs(g12 - st["G12"]) <= tl.STAT_RTOL * ab[2] + 1e-37)
                    ok, _, plain = tl.rel_close(A[b, h, off:off + 2 * P].cpu().numpy(), st["A"][off:off + 2 * P])
                    assert ok, plain
                    ok, nm, nout = tl.mask_band_ok(mask[b, h, :P].cpu().numpy(), st["mask"], st["score"], st["R"])
                    assert ok, (nm, nout)
                    c12 = st["G12"] if mode == 1 else 0.0
                    gam = st["G11"] + 2.0 * c12 + st["G22"]
                    tot = ab[0] + ab[1] + (2.0 * ab[2] if mode == 1 else 0.0)
                    dw = np.abs(wg[b, h, :P].cpu().numpy() - st["w"])
                    clear = np.abs(gam) > 1e-3 * tot            # away from the guard on the denominator
                    bound = np.minimum(1.0, tl.STAT_RTOL * tot / np.maximum(np.abs(gam), 1e-300)) + 1e-7
                    assert np.all(dw[clear] <= bound[clear]), float(np.max((dw / bound)[clear]))
                    assert clear.mean() > 0.95
                    n_ratio += int(np.sum((st["w"] > 0) & (st["w"] < 1) & (st["w"] != 0.5)))
            assert n_ratio > 50
    # the whole pass with exact weights on a fresh small cache
    # (seed chosen so that no merged pair sits near the guard of its denominator)
    w2 = _small(seed=76, batch=1, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(500,), budgets=(140,))
    d2 = wl.make_layer(w2)
    E2 = wl.f32_to_bf16_bits(np.random.default_rng(76).standard_normal(d2["q_win"].shape).astype(np.float32))
    for mode in (1, 2):
        *_, flips = full_pass_vs_oracle(kb, w2, d2, exact=(E2, mode))


def test_merge_pass_replayed_from_a_cuda_graph(kb):
    """The merge pass and the decode check, captured once into a CUDA graph and replayed twice on
    a restored cache, must give bit for bit what the same calls gave when launched directly:
    everything a call needs on the device travels as kernel arguments or lives in the caller's
    workspace, nothing depends on host work at launch time."""
    import torch
    w = _small(seed=31, seq_lens=(700, 389), budgets=(256, 120), n_decode=4)
    data = wl.make_layer(w)
    dev, p, ws = _setup(kb, w, data)
    B, Hq, T = w.batch, w.n_q_heads, w.n_decode
    K0, V0, C0 = dev["K"].clone(), dev["V"].clone(), dev["counts"].clone()
    out = torch.zeros((B, Hq, T, 128), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def restore():
        dev["K"].copy_(K0); dev["V"].copy_(V0); dev["counts"].copy_(C0); out.zero_()

    def run():
        new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                                     list(w.budgets), ws, status_dev=status)
        kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], new_len, out, ws)
        return new_len

    # launched directly (also the first call on this device, outside any capture)
    new_len = run()
    torch.cuda.synchronize()
    assert status.item() == 0 and new_len == list(w.budgets)
    ref = [tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy(), tl.bits_of(out)]
    # once more on a side stream, then the capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        restore(); run()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    restore()
    with torch.cuda.graph(graph):
        assert run() == new_len
    for _ in range(2):
        restore()
        graph.replay()
        torch.cuda.synchronize()
        assert status.item() == 0
        got = [tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy(), tl.bits_of(out)]
        for b in range(B):
            m = new_len[b]
            for g, r in zip(got[:3], ref[:3]):
                assert np.array_equal(g[b, :, :m], r[b, :, :m])
        assert np.array_equal(got[3], ref[3])


def test_repeated_passes_are_bit_identical(kb):
    """The same batch merged twenty times from the same start gives the same bits every time (partial
    sums are added in a fixed order, no atomics on data), also when the calls follow one another on
    the stream without a host synchronisation in between: the kernels of one pass start while their
    predecessors drain, and a kernel that read too early would show up here as a changed result."""
    import torch
    w = _small(seed=91, batch=3, n_q_heads=8, n_kv_heads=2, window=16, seq_lens=(1500, 900, 333),
               budgets=(400, 300, 333), n_decode=3)
    data = wl.make_layer(w)
    dev, p, ws = _setup(kb, w, data)
    B, Hq, T = w.batch, w.n_q_heads, w.n_decode
    K0, V0, C0 = dev["K"].clone(), dev["V"].clone(), dev["counts"].clone()
    outs = [torch.zeros((B, Hq, T, 128), dtype=torch.bfloat16, device="cuda") for _ in range(20)]
    snaps = []
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for it in range(20):
        dev["K"].copy_(K0); dev["V"].copy_(V0); dev["counts"].copy_(C0)
        new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                                     list(w.budgets), ws, status_dev=status)
        kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], new_len, outs[it], ws)
        snaps.append((dev["K"].clone(), dev["V"].clone(), dev["counts"].clone()))   # (stream ordered, no sync)
    torch.cuda.synchronize()
    assert status.item() == 0 and new_len == [400, 300, 333]
    for it in range(1, 20):
        for b in range(B):
            m = new_len[b]
            for x, y in zip(snaps[it], snaps[0]):
                assert torch.equal(x[b, :, :m], y[b, :, :m]), (it, b)
        assert torch.equal(outs[it], outs[0]), it
