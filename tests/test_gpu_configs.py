"""Parity at the full shape of every benchmark configuration, in the launch shapes the benchmark
uses (layers folded into the batch).  The oracle cannot redo whole layers of the large ones inside
a test, so each case checks sampled (sequence, KV head) units element by element, integer work
(selection over the GPU's own scores, compaction) bit for bit at full size, and properties that
hold for every unit."""
import math

import numpy as np
import pytest

from oracle import kvs_oracle as oc
from paper_2603_00907_b200 import workloads as wl
from tests import kvs_testlib as tl
from tests import test_gpu_parity as tp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kb():
    from paper_2603_00907_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _fold(w, layers, n_decode):
    """Layers folded into the batch dimension, as the benchmark passes them."""
    per_layer = wl.make_layers_parallel(w.scaled(n_decode=n_decode), layers)
    data = {k: np.concatenate([d[k] for d in per_layer], axis=0) for k in ("K", "V", "counts", "q_win", "q_new")}
    L = len(per_layer)
    folded = w.scaled(batch=w.batch * L, seq_lens=tuple(w.seq_lens) * L, budgets=tuple(w.budgets) * L,
                      n_decode=n_decode)
    return folded, data


def _oracle_stats(w, data, b, h, r=0):
    n, G = int(w.seq_lens[b]), w.group
    return oc.round_stats(data["K"][b, h, :n], data["V"][b, h, :n], data["counts"][b, h, :n].astype(np.int64),
                          data["q_win"][b, h * G:(h + 1) * G], w.budgets[b], r, window=w.window, sink=w.sink,
                          recent=w.window, scale=1 / math.sqrt(128), causal=True, round_frac=w.round_frac,
                          score_mode=0)


def _round0_stats_of_units(kb, w, data, units):
    """kvs_window_stats over the whole batch; sampled units against the oracle."""
    import torch
    dev, p, ws = tp._setup(kb, w, data)
    B, Hkv, Nmax = data["K"].shape[:3]
    f32 = dict(dtype=torch.float32, device="cuda")
    A, N1 = torch.zeros((B, Hkv, Nmax), **f32), torch.zeros((B, Hkv, Nmax), **f32)
    N12, score, wgt, cosv = (torch.zeros((B, Hkv, Nmax // 2), **f32) for _ in range(4))
    mask = torch.zeros((B, Hkv, Nmax // 2), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kb.kvs_window_stats(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens), list(w.budgets), ws,
                        A=A, N1=N1, N12=N12, cosv=cosv, score=score, w=wgt, mask=mask, status_dev=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for (b, h) in units:
        st = _oracle_stats(w, data, b, h)
        got = {"A": A[b, h].cpu().numpy(), "N1": N1[b, h].cpu().numpy(), "N12": N12[b, h].cpu().numpy(),
               "cos": cosv[b, h].cpu().numpy(), "score": score[b, h].cpu().numpy(), "w": wgt[b, h].cpu().numpy(),
               "mask": mask[b, h].cpu().numpy()}
        tl.check_unit_stats(got, st, label=f"unit {(b, h)}")
    return dev, p, ws


def _properties_of_merged_cache(w, data, Kg, Vg, Cg, new_len):
    """What holds for every unit after the pass: the budget is met, every token is still counted,
    the protected prefix and suffix are untouched, value sums are conserved up to bf16 rounding."""
    B, Hkv = data["K"].shape[:2]
    for b in range(B):
        n, m = int(w.seq_lens[b]), new_len[b]
        assert m == min(n, w.budgets[b])
        for h in range(Hkv):
            c = Cg[b, h, :m]
            assert int(c.sum()) == n and c.min() >= 1
            assert np.array_equal(Kg[b, h, :w.sink], data["K"][b, h, :w.sink])
            assert np.array_equal(Kg[b, h, m - w.window:m], data["K"][b, h, n - w.window:n])
            assert np.array_equal(Vg[b, h, m - w.window:m], data["V"][b, h, n - w.window:n])
            assert np.all(c[:w.sink] == 1) and np.all(c[m - w.window:] == 1)
            tot = oc.bf16_to_f64(data["V"][b, h, :n]).sum(0)
            got = oc.bf16_to_f64(Vg[b, h, :m]).sum(0)
            assert np.max(np.abs(got - tot)) < 0.02 * math.sqrt(n)      # bf16 roundings of ~n merges


def _decode_of_units(kb, w, data, dev, p, ws, new_len, units):
    import torch
    B, T = data["K"].shape[0], data["q_new"].shape[2]
    G = w.group
    out = torch.zeros((B, w.n_q_heads, T, 128), dtype=torch.bfloat16, device="cuda")
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], new_len, out, ws)
    torch.cuda.synchronize()
    og = tl.bits_of(out)
    Kg, Vg, Cg = tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy()
    for (b, h) in units:
        m = new_len[b]
        ref, _ = oc.decode_attention(data["q_new"][b, h * G:(h + 1) * G], Kg[b, h, :m], Vg[b, h, :m], Cg[b, h, :m])
        ok, mx, _, _ = tl.bf16_close(og[b, h * G:(h + 1) * G], oc.f64_to_bf16(ref))
        assert ok, ((b, h), mx)
    return Kg, Vg, Cg


def test_config0_whole_layer_against_the_oracle(kb):
    """configs[0]: one layer, 4096 tokens, 8 KV heads, 4 x 32 window rows, budget 1024: every unit
    through all five rounds against the oracle that follows the GPU's in-band choices."""
    w = wl.config(0)
    data = wl.make_layer(w, 0)
    _, _, _, new_len, flips = tp.full_pass_vs_oracle(kb, w, data)
    assert new_len == [1024]
    print(f"configs[0]: band flips followed: {flips}")


def test_config1_sampled_unit_through_all_rounds(kb):
    """configs[1] shape (32768 tokens, 4 x 64 window rows, budget 2048), five layers folded into the
    batch: one sampled unit through all ten rounds against the oracle; every unit's bookkeeping."""
    w, data = _fold(wl.config(1), range(5), 1)
    Kg, Vg, Cg, new_len, flips = tp.full_pass_vs_oracle(kb, w, data, units=[(3, 5)])
    _properties_of_merged_cache(w, data, Kg, Vg, Cg, new_len)
    print(f"configs[1]: band flips followed: {flips}")


def test_config2_qwen_layout_all_layers_folded(kb):
    """configs[2]: 28 layers x 4 sequences of 16384 tokens folded into 112 sequences, 4 KV heads,
    7 x 32 = 224 window rows (a partial second query block), budget 1024."""
    import torch
    w, data = _fold(wl.config(2), range(28), 1)
    units = [(0, 0), (77, 3)]
    dev, p, ws = _round0_stats_of_units(kb, w, data, units)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                                 list(w.budgets), ws, status_dev=status)
    Kg, Vg, Cg = _decode_of_units(kb, w, data, dev, p, ws, new_len, [(5, 1), (111, 2)])
    assert status.item() == 0
    _properties_of_merged_cache(w, data, Kg, Vg, Cg, new_len)


def test_config3_ragged_batch_with_decode(kb):
    """configs[3]: eight sequences of 4096-65536 tokens, budgets of 12.5 %, 32 new query tokens per
    sequence for the decode check.  Statistics of the longest and the shortest sequence."""
    import torch
    w = wl.config(3)
    data = wl.make_layer(w, 0)
    longest, shortest = int(np.argmax(w.seq_lens)), int(np.argmin(w.seq_lens))
    dev, p, ws = _round0_stats_of_units(kb, w, data, [(longest, 2), (shortest, 6)])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                                 list(w.budgets), ws, status_dev=status)
    assert new_len == [n // 8 for n in w.seq_lens]
    Kg, Vg, Cg = _decode_of_units(kb, w, data, dev, p, ws, new_len, [(longest, 0), (shortest, 7), (3, 4)])
    assert status.item() == 0
    _properties_of_merged_cache(w, data, Kg, Vg, Cg, new_len)


def test_config4_statistics_on_sampled_slots_and_exact_selection(kb):
    """configs[4]: 131072 tokens, 8 x 128 = 1024 window rows (eight query blocks), budget 4096.
    The oracle forms the window probabilities of one unit once and the per-slot / per-pair
    statistics on a sample of candidate pairs; the selection is checked at full size as integer
    work on the GPU's own scores (the R smallest (score, index)), and on the sample against the
    oracle's scores modulo the cutoff band."""
    import torch
    w = wl.config(4)
    data = wl.make_layer(w.scaled(n_decode=1), 0)
    n, bud, G, W = w.seq_lens[0], w.budgets[0], w.group, w.window
    dev, p, ws = tp._setup(kb, w.scaled(n_decode=1), data)
    Hkv, Nmax = w.n_kv_heads, w.n_max
    f32 = dict(dtype=torch.float32, device="cuda")
    A, N1 = torch.zeros((1, Hkv, Nmax), **f32), torch.zeros((1, Hkv, Nmax), **f32)
    N12, score, wgt, cosv = (torch.zeros((1, Hkv, Nmax // 2), **f32) for _ in range(4))
    mask = torch.zeros((1, Hkv, Nmax // 2), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kb.kvs_window_stats(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [n], [bud], ws, A=A, N1=N1, N12=N12,
                        cosv=cosv, score=score, w=wgt, mask=mask, status_dev=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    off, P, R = oc.round_plan(n, bud, w.sink, W, w.round_frac, 0)
    # selection, all heads, bit for bit: the R smallest (score bits, index) of the GPU's own scores
    for h in range(Hkv):
        sg = score[0, h, :P].cpu().numpy()
        assert np.array_equal(mask[0, h, :P].cpu().numpy(), oc.select_pairs(sg.astype(np.float64), R))
    # one unit: probabilities once, statistics on 1500 sampled candidate pairs
    h = 5
    Kf, Vf = oc.bf16_to_f64(data["K"][0, h, :n]), oc.bf16_to_f64(data["V"][0, h, :n])
    Qf = oc.bf16_to_f64(data["q_win"][0, h * G:(h + 1) * G])
    alpha, o, vbar = oc.window_probabilities(Kf, Vf, np.ones(n), Qf, W, 1 / math.sqrt(128), True)
    rng = np.random.default_rng(4)
    pairs = np.sort(rng.choice(P, size=1500, replace=False))
    pairs[:3], pairs[-3:] = (0, 1, 2), (P - 3, P - 2, P - 1)       # first and last candidates included
    pairs = np.unique(pairs)
    idx = np.stack([off + 2 * pairs, off + 2 * pairs + 1], axis=1).reshape(-1)
    a_s, v_s = np.ascontiguousarray(alpha[:, idx]), vbar[idx]
    del alpha
    A_s, N1_s = oc.slot_stats(a_s, o, v_s)
    N12_s, cos_s, score_s = oc.pair_stats(Kf[idx], a_s, o, v_s, A_s, 0, len(pairs), 0)
    w_s = oc.pair_weights(N1_s, N12_s, 0, len(pairs))
    got = {"A": A[0, h].cpu().numpy()[idx], "N1": N1[0, h].cpu().numpy()[idx],
           "N12": N12[0, h].cpu().numpy()[pairs], "cos": cosv[0, h].cpu().numpy()[pairs],
           "score": score[0, h].cpu().numpy()[pairs], "w": wgt[0, h].cpu().numpy()[pairs]}
    ref = {"off": 0, "P": len(pairs), "A": A_s, "N1": N1_s, "N12": N12_s, "cos": cos_s, "score": score_s, "w": w_s}
    tl.check_unit_stats(got, ref, label="configs[4] sampled pairs", with_mask=False)
    # the GPU's decision on the sampled pairs against the oracle's scores: away from the GPU's cutoff
    # (by more than the band) the two must agree
    sg = score[0, h, :P].cpu().numpy().astype(np.float64)
    cutoff = np.sort(sg)[R - 1]
    mg = mask[0, h].cpu().numpy()[pairs]
    clear = np.abs(score_s - cutoff) > tl.MASK_BAND * cutoff
    assert np.array_equal(mg[clear], (score_s[clear] < cutoff).astype(np.uint8))
    assert clear.mean() > 0.99


def test_config4_compaction_at_full_length_bit_exact(kb):
    """kvs_compact on 131072-slot units with random valid decisions: 37 persistent CTAs per unit
    hand rows to one another through the "tile loaded" flags.  Indices, counts and value sums bit
    for bit, keys within one bf16 ulp, both pair parities."""
    import torch
    w = wl.config(4)
    data = wl.make_layer(w, 0)
    rng = np.random.default_rng(44)
    Hkv, Nmax = w.n_kv_heads, w.n_max
    K, V, C = data["K"], data["V"], data["counts"]
    Kd, Vd, Cd = tl.to_dev_bf16(K), tl.to_dev_bf16(V), torch.from_numpy(C).cuda()
    n = w.seq_lens[0]
    for r, frac in ((0, 0.5), (1, 0.03)):
        off = w.sink + (r % 2)
        P = (n - off - w.window) // 2
        R = int(frac * P)
        mask = np.zeros((1, Hkv, Nmax // 2), dtype=np.uint8)
        wgt = rng.random((1, Hkv, Nmax // 2), dtype=np.float32)
        for h in range(Hkv):
            mask[0, h, rng.choice(P, size=R, replace=False)] = 1
        p = kb.make_params(Kd, Vd, w.n_q_heads, w.window, sink=w.sink, first_round=r)
        ws = torch.empty(kb.kvs_workspace_size(p, Nmax, 0), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        new_index = torch.full((1, Hkv, Nmax), -1, dtype=torch.int32, device="cuda")
        got = kb.kvs_compact(p, Kd, Vd, Cd, torch.from_numpy(mask).cuda(), torch.from_numpy(wgt).cuda(), [n], [R], ws,
                             new_index=new_index, status_dev=status)
        torch.cuda.synchronize()
        assert status.item() == 0 and got == [n - R]
        Kg, Vg, Cg, ig = tl.bits_of(Kd), tl.bits_of(Vd), Cd.cpu().numpy(), new_index.cpu().numpy()
        m = n - R
        Kn, Vn, Cn = np.zeros_like(K), np.zeros_like(V), np.zeros_like(C)
        for h in range(Hkv):
            k2, v2, c2, ix = oc.apply_merge(K[0, h, :n], V[0, h, :n], C[0, h, :n].astype(np.int64), off,
                                            mask[0, h, :P], wgt[0, h, :P].astype(np.float64))
            Kn[0, h, :m], Vn[0, h, :m], Cn[0, h, :m] = k2, v2, c2
            assert np.array_equal(Cg[0, h, :m], c2)
            assert np.array_equal(ig[0, h, :n], ix)
            assert np.array_equal(Vg[0, h, :m], v2)
            ok, mx, nulp, worse = tl.bf16_close(Kg[0, h, :m], k2, atol=0.0)
            assert ok, (mx, nulp, worse)
        K, V, C, n = Kn, Vn, Cn, m


def test_config4_full_pass_and_split_decode(kb):
    """configs[4] end to end: thirteen rounds from 131072 to 4096 slots, then decode attention of
    new tokens over the merged cache against the oracle's attention over the same cache."""
    import torch
    w = wl.config(4)
    data = wl.make_layer(w, 0)
    dev, p, ws = tp._setup(kb, w, data)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                                 list(w.budgets), ws, status_dev=status)
    assert new_len == [4096]
    Kg, Vg, Cg = _decode_of_units(kb, w, data, dev, p, ws, new_len, [(0, 1), (0, 6)])
    assert status.item() == 0
    _properties_of_merged_cache(w, data, Kg, Vg, Cg, new_len)
