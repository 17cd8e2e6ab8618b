"""Failure and padding paths of the CUDA kernels, exercised without any fault or real stall.

* Bounded waits: with the library's test hook one kind of wait is left without its signal (the
  producer requests no K tiles; the compaction publishes no "tile loaded" flags) and the time limit
  is shortened to a few milliseconds.  The kernel must return by itself with KVS_ERR_TIMEOUT in
  *status_dev, and the next ordinary call on the same stream must pass its parity check.
* Padding: rows and counts behind seq_len hold NaN, infinities and random bit patterns; every
  result must be bit-identical to the run on a zero-padded cache.
* Small edge cases of the boundary: sequences that end inside the protected prefix, an odd
  capacity without a protected suffix.
"""
import math

import numpy as np
import pytest

from oracle import kvs_oracle as oc
from paper_2603_00907_b200 import workloads as wl
from tests import kvs_testlib as tl
from tests import test_gpu_parity as tp

pytestmark = pytest.mark.gpu

KVS_ERR_TIMEOUT = 6
LIMIT_US = 3000


@pytest.fixture(scope="module")
def kb():
    from paper_2603_00907_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def test_attention_wait_runs_out_then_the_next_call_is_clean(kb):
    import torch
    w = tp._small(seed=41, batch=1, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(600,), budgets=(600,), n_decode=4)
    data = wl.make_layer(w)
    dev, p, ws = tp._setup(kb, w, data)
    out = torch.zeros((1, w.n_q_heads, 4, 128), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kb.kvs_debug_set_wait(LIMIT_US, 1)
    try:
        kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], [600], out, ws, status_dev=status)
        torch.cuda.synchronize()
    finally:
        kb.kvs_debug_set_wait(0, 0)
    assert status.item() == KVS_ERR_TIMEOUT
    status.zero_()
    kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], [600], out, ws, status_dev=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    G = w.group
    for h in range(w.n_kv_heads):
        ref, _ = oc.decode_attention(data["q_new"][0, h * G:(h + 1) * G], data["K"][0, h, :600], data["V"][0, h, :600],
                                     data["counts"][0, h, :600])
        ok, mx, _, _ = tl.bf16_close(tl.bits_of(out)[0, h * G:(h + 1) * G], oc.f64_to_bf16(ref))
        assert ok, mx


def test_statistics_wait_runs_out_then_the_next_call_is_clean(kb):
    import torch
    w = tp._small(seed=42, batch=1, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(900,), budgets=(300,))
    data = wl.make_layer(w)
    dev, p, ws = tp._setup(kb, w, data)
    score = torch.zeros((1, 2, w.n_max // 2), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kb.kvs_debug_set_wait(LIMIT_US, 2)
    try:
        kb.kvs_window_stats(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [900], [300], ws, score=score,
                            status_dev=status)
        torch.cuda.synchronize()
    finally:
        kb.kvs_debug_set_wait(0, 0)
    assert status.item() == KVS_ERR_TIMEOUT
    tp._check_round_stats(kb, w, data["K"], data["V"], data["counts"], data["q_win"], [900], 0)


def test_compaction_flag_wait_runs_out_then_the_next_call_is_clean(kb):
    import torch
    w = tp._small(seed=43, batch=1, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(4000,), budgets=(1000,))
    data = wl.make_layer(w)
    rng = np.random.default_rng(43)
    Hkv, Nmax, n = w.n_kv_heads, w.n_max, 4000
    off = w.sink
    P = (n - off - w.window) // 2
    R = P // 3
    mask = np.zeros((1, Hkv, Nmax // 2), dtype=np.uint8)
    wgt = rng.random((1, Hkv, Nmax // 2), dtype=np.float32)
    for h in range(Hkv):
        mask[0, h, rng.choice(P, size=R, replace=False)] = 1
    dm, dw = torch.from_numpy(mask).cuda(), torch.from_numpy(wgt).cuda()
    dev, p, ws = tp._setup(kb, w, data)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kb.kvs_debug_set_wait(LIMIT_US, 4)
    try:
        kb.kvs_compact(p, dev["K"], dev["V"], dev["counts"], dm, dw, [n], [R], ws, status_dev=status)
        torch.cuda.synchronize()
    finally:
        kb.kvs_debug_set_wait(0, 0)
    assert status.item() == KVS_ERR_TIMEOUT
    # a fresh copy of the cache through the same entry point: bit for bit against the oracle's bookkeeping
    dev, p, ws = tp._setup(kb, w, data)
    status.zero_()
    new_index = torch.full((1, Hkv, Nmax), -1, dtype=torch.int32, device="cuda")
    got = kb.kvs_compact(p, dev["K"], dev["V"], dev["counts"], dm, dw, [n], [R], ws, new_index=new_index,
                         status_dev=status)
    torch.cuda.synchronize()
    assert status.item() == 0 and got == [n - R]
    for h in range(Hkv):
        k2, v2, c2, ix = oc.apply_merge(data["K"][0, h, :n], data["V"][0, h, :n], data["counts"][0, h, :n].astype(np.int64),
                                        off, mask[0, h, :P], wgt[0, h, :P].astype(np.float64))
        assert np.array_equal(dev["counts"].cpu().numpy()[0, h, :n - R], c2)
        assert np.array_equal(new_index.cpu().numpy()[0, h, :n], ix)
        assert np.array_equal(tl.bits_of(dev["V"])[0, h, :n - R], v2)
        ok, mx, _, worse = tl.bf16_close(tl.bits_of(dev["K"])[0, h, :n - R], k2, atol=0.0)
        assert ok, (mx, worse)


def _poison(data, seq_lens, rng):
    """Copies of K, V, counts whose rows at or behind seq_len[b] hold NaN, infinities and random bits."""
    K, V, C = data["K"].copy(), data["V"].copy(), data["counts"].copy()
    patterns = np.array([0x7FC0, 0xFFC0, 0x7F80, 0xFF80, 0x7FFF, 0x7F7F, 0xFF7F], dtype=np.uint16)
    for b, n in enumerate(seq_lens):
        tail = K[b, :, n:].shape
        K[b, :, n:] = np.where(rng.random(tail) < 0.7, rng.choice(patterns, size=tail),
                               rng.integers(0, 1 << 16, size=tail).astype(np.uint16))
        V[b, :, n:] = np.where(rng.random(tail) < 0.7, rng.choice(patterns, size=tail),
                               rng.integers(0, 1 << 16, size=tail).astype(np.uint16))
        C[b, :, n:] = rng.integers(-(1 << 31), (1 << 31) - 1, size=C[b, :, n:].shape, dtype=np.int64).astype(np.int32)
    return K, V, C


def test_garbage_behind_seq_len_changes_nothing(kb):
    """A ragged batch in a padded layout: what lies behind a sequence's last slot (up to the shared
    capacity, which also pads the last tiles) must not reach any result."""
    import torch
    w = tp._small(seed=44, batch=4, n_q_heads=8, n_kv_heads=2, window=16, seq_lens=(1201, 300, 77, 1000),
                  budgets=(150, 64, 77, 125), n_decode=3)
    data = wl.make_layer(w)
    rng = np.random.default_rng(9)
    Kp, Vp, Cp = _poison(data, w.seq_lens, rng)
    assert np.isnan(oc.bf16_to_f64(Kp[1, 0, 300:])).any()
    B, Hkv, Nmax, M = w.batch, w.n_kv_heads, w.n_max, w.group * w.window
    results = []
    for K, V, C in ((data["K"], data["V"], data["counts"]), (Kp, Vp, Cp)):
        dev, p, ws = tp._setup(kb, w, {**data, "K": K, "V": V, "counts": C})
        f32 = dict(dtype=torch.float32, device="cuda")
        A, N1 = torch.zeros((B, Hkv, Nmax), **f32), torch.zeros((B, Hkv, Nmax), **f32)
        N12, cosv, score, wgt = (torch.zeros((B, Hkv, Nmax // 2), **f32) for _ in range(4))
        mask = torch.zeros((B, Hkv, Nmax // 2), dtype=torch.uint8, device="cuda")
        o_win, lse = torch.zeros((B, Hkv, M, 128), **f32), torch.zeros((B, Hkv, M), **f32)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for r in (0, 1):
            pr = kb.make_params(dev["K"], dev["V"], w.n_q_heads, w.window, sink=w.sink, first_round=r)
            kb.kvs_window_stats(pr, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens), list(w.budgets),
                                ws, A=A, N1=N1, N12=N12, cosv=cosv, score=score, w=wgt, mask=mask, o_win=o_win,
                                lse_win=lse, status_dev=status)
            torch.cuda.synchronize()
            results.append([t.cpu().numpy().copy() for t in (A, N1, N12, cosv, score, wgt, mask, o_win, lse)])
        out0 = torch.zeros((B, w.n_q_heads, 3, 128), dtype=torch.bfloat16, device="cuda")
        kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], list(w.seq_lens), out0, ws,
                           status_dev=status)
        new_len = kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], list(w.seq_lens),
                                     list(w.budgets), ws, status_dev=status)
        out1 = torch.zeros_like(out0)
        kb.kvs_decode_attn(p, dev["q_new"], dev["K"], dev["V"], dev["counts"], new_len, out1, ws, status_dev=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        Kg, Vg, Cg = tl.bits_of(dev["K"]), tl.bits_of(dev["V"]), dev["counts"].cpu().numpy()
        results.append([tl.bits_of(out0), tl.bits_of(out1)] +
                       [x[b, :, :new_len[b]].copy() for b in range(B) for x in (Kg, Vg, Cg)])
    half = len(results) // 2
    for clean, dirty in zip(results[:half], results[half:]):
        for x, y in zip(clean, dirty):
            assert np.array_equal(x, y, equal_nan=True)
    assert not np.isnan(results[half][0]).any()


def test_sequences_inside_the_protected_prefix_get_the_identity_map(kb):
    import torch
    w = tp._small(seed=45, batch=3, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(20, 300, 32), budgets=(20, 100, 32))
    data = wl.make_layer(w)
    dev, p, ws = tp._setup(kb, w, data)
    B, Hkv, Nmax = w.batch, w.n_kv_heads, w.n_max
    rng = np.random.default_rng(45)
    P = (300 - w.sink - w.window) // 2
    mask = np.zeros((B, Hkv, Nmax // 2), dtype=np.uint8)
    for h in range(Hkv):
        mask[1, h, rng.choice(P, size=40, replace=False)] = 1
    wgt = rng.random((B, Hkv, Nmax // 2), dtype=np.float32)
    new_index = torch.full((B, Hkv, Nmax), -1, dtype=torch.int32, device="cuda")
    got = kb.kvs_compact(p, dev["K"], dev["V"], dev["counts"], torch.from_numpy(mask).cuda(), torch.from_numpy(wgt).cuda(),
                         [20, 300, 32], [0, 40, 0], ws, new_index=new_index)
    torch.cuda.synchronize()
    ni = new_index.cpu().numpy()
    assert got == [20, 260, 32]
    for b, n in ((0, 20), (2, 32)):
        assert np.array_equal(ni[b, :, :n], np.tile(np.arange(n, dtype=np.int32), (Hkv, 1)))
        assert np.all(ni[b, :, n:] == -1)
        assert np.array_equal(tl.bits_of(dev["K"])[b], data["K"][b])
    for h in range(Hkv):
        _, _, _, ix = oc.apply_merge(data["K"][1, h, :300], data["V"][1, h, :300], data["counts"][1, h, :300].astype(np.int64),
                                     w.sink, mask[1, h, :P], wgt[1, h, :P].astype(np.float64))
        assert np.array_equal(ni[1, h, :300], ix)


def test_odd_capacity_without_protected_suffix_is_refused(kb):
    import torch
    w = tp._small(seed=46, batch=1, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(301,), budgets=(100,))
    data = wl.make_layer(w)
    dev = tl.upload_layer(data)
    p = kb.make_params(dev["K"], dev["V"], w.n_q_heads, w.window, sink=w.sink, recent=0, causal=False)
    ws = torch.empty(kb.kvs_workspace_size(p, w.n_max, 0), dtype=torch.uint8, device="cuda")
    before = tl.bits_of(dev["K"]).copy()
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_merge_layer(p, dev["K"], dev["V"], dev["counts"], dev["q_win"], [301], [100], ws)
    assert e.value.code == 2
    torch.cuda.synchronize()
    assert np.array_equal(tl.bits_of(dev["K"]), before)
    # with one protected trailing slot the same capacity is fine
    p1 = kb.make_params(dev["K"], dev["V"], w.n_q_heads, w.window, sink=w.sink, recent=1, causal=False)
    assert kb.kvs_merge_layer(p1, dev["K"], dev["V"], dev["counts"], dev["q_win"], [301], [100], ws) == [100]
    torch.cuda.synchronize()


def test_operand_feed_probe_reports_sane_cycles(kb):
    """The tensor-core operand-feed probe ends by itself and reports what the arithmetic allows at
    the least: a 128 x 256 x 16 product cannot take fewer than 128 cycles (4096 multiply-adds per
    cycle), a 128 x 64 x 16 one not fewer than 32; taking the A slice from the collector buffer
    for every second product must not make the narrow products slower."""
    import torch
    blocks, products = 4, 512
    out = {}
    for n_cols, reuse in ((256, False), (64, False), (64, True)):
        cyc = torch.zeros(blocks, dtype=torch.int64, device="cuda")
        kb.kvs_probe_mma(blocks, n_cols, reuse, products, cyc)
        torch.cuda.synchronize()
        c = cyc.cpu().numpy()
        assert (c > 0).all(), c
        out[(n_cols, reuse)] = c.max() / products
    assert 120 <= out[(256, False)] < 400, out
    assert 30 <= out[(64, False)] < 200, out
    assert out[(64, True)] <= out[(64, False)] * 1.05, out
