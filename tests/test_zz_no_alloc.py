"""kvs_compact_static: the compaction for callers that cannot allocate device memory (an engine
that owns all of the GPU's memory, a section where cudaMalloc's implicit synchronisation is not
acceptable).  Its scratch is a fixed array inside the library, so the test checks that it gives
exactly what kvs_compact gives with a caller-made workspace - twice in a row, because the second
call finds the array as the first one left it."""
import numpy as np
import pytest

from paper_2603_00907_b200 import workloads as wl
from tests import kvs_testlib as tl

pytestmark = pytest.mark.gpu


def _random_decision(rng, w, n_list, r):
    """A valid merge decision: per sequence the same number of pairs in every head."""
    B, Hkv, Nmax = w.batch, w.n_kv_heads, w.n_max
    off = w.sink + (r % 2)
    mask = np.zeros((B, Hkv, Nmax // 2), dtype=np.uint8)
    wgt = rng.random((B, Hkv, Nmax // 2), dtype=np.float32)
    n_merge = []
    for b in range(B):
        P = max(0, (n_list[b] - off - w.window) // 2)
        R = int(rng.integers(1, max(2, P // 2)))
        for h in range(Hkv):
            mask[b, h, rng.choice(P, size=R, replace=False)] = 1
        n_merge.append(R)
    return mask, wgt, n_merge


def test_static_scratch_compaction_equals_workspace_compaction_twice():
    import torch
    from paper_2603_00907_b200 import binding as kb, build
    build.build()
    w = wl.small_case(21, batch=2, n_q_heads=8, n_kv_heads=2, window=8, seq_lens=(700, 413),
                      budgets=(100, 100))
    data = wl.make_layer(w)
    rng = np.random.default_rng(7)
    a, b = tl.upload_layer(data), tl.upload_layer(data)          # two copies of the same cache
    B, Hkv, Nmax = w.batch, w.n_kv_heads, w.n_max
    n_list = list(w.seq_lens)
    assert kb.kvs_static_scratch_bytes() == 4 << 20
    for r in (0, 1):                                             # two calls in a row
        mask, wgt, n_merge = _random_decision(rng, w, n_list, r)
        dm, dw = torch.from_numpy(mask).cuda(), torch.from_numpy(wgt).cuda()
        p = kb.make_params(a["K"], a["V"], w.n_q_heads, w.window, sink=w.sink, first_round=r)
        ws = torch.empty(kb.kvs_workspace_size(p, Nmax, 0), dtype=torch.uint8, device="cuda")
        ia = torch.full((B, Hkv, Nmax), -1, dtype=torch.int32, device="cuda")
        ib = torch.full((B, Hkv, Nmax), -1, dtype=torch.int32, device="cuda")
        sa = torch.zeros(1, dtype=torch.int32, device="cuda")
        sb = torch.zeros(1, dtype=torch.int32, device="cuda")
        len_a = kb.kvs_compact(p, a["K"], a["V"], a["counts"], dm, dw, n_list, n_merge, ws,
                               new_index=ia, status_dev=sa)
        torch.cuda.synchronize()
        len_b = kb.kvs_compact_static(p, b["K"], b["V"], b["counts"], dm, dw, n_list, n_merge,
                                      new_index=ib, status_dev=sb)
        torch.cuda.synchronize()
        assert sa.item() == 0 and sb.item() == 0
        assert len_a == len_b == [n - m for n, m in zip(n_list, n_merge)]
        for s in range(B):
            m, n = len_a[s], n_list[s]
            # integer work and fp32 arithmetic on identical inputs: bit for bit
            assert np.array_equal(tl.bits_of(a["K"])[s, :, :m], tl.bits_of(b["K"])[s, :, :m])
            assert np.array_equal(tl.bits_of(a["V"])[s, :, :m], tl.bits_of(b["V"])[s, :, :m])
            assert np.array_equal(a["counts"].cpu().numpy()[s, :, :m], b["counts"].cpu().numpy()[s, :, :m])
            assert np.array_equal(ia.cpu().numpy()[s, :, :n], ib.cpu().numpy()[s, :, :n])
            assert int(b["counts"].cpu().numpy()[s, 0, :m].sum()) == w.seq_lens[s]
        n_list = len_a


def test_static_scratch_rejects_what_does_not_fit():
    import torch
    from paper_2603_00907_b200 import binding as kb, build
    build.build()
    # 64 units x 2^20 slots would need 8 MiB of scratch; nothing is dereferenced before the check
    B, Hkv, Nmax = 8, 8, 1 << 20
    p = kb.kvs_params_t()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = B, 32, Hkv, 128
    p.window, p.sink, p.recent, p.causal = 32, 32, 32, 1
    p.softmax_scale, p.round_frac, p.score_mode, p.first_round = 128 ** -0.5, 0.5, 0, 0
    p.k_stride_t = p.v_stride_t = 128
    p.k_stride_h = p.v_stride_h = 128 * Nmax
    p.k_stride_b = p.v_stride_b = 128 * Nmax * Hkv
    tiny = torch.zeros(64, dtype=torch.uint8, device="cuda")     # stands in for every pointer

    class Shape:                                                 # counts.shape[-1] is n_max
        shape = (B, Hkv, Nmax)

        @staticmethod
        def data_ptr():
            return tiny.data_ptr()

    with pytest.raises(kb.KvsError) as e:
        kb.kvs_compact_static(p, tiny, tiny, Shape, tiny, tiny, [1000] * B, [1] * B)
    assert e.value.code == 3 and "kvs_compact_static" in str(e.value)
