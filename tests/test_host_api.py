"""Host-side checks that need no GPU: the library loads, exports every declared symbol,
its round scheduler matches the oracle's schedule, and argument errors are reported."""
import ctypes
import os
import re

import pytest

from oracle import kvs_oracle as oc
from paper_2603_00907_b200 import binding as kb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2603_00907_b200 import build
    build.build()
    return kb.lib()


def _params(**kw):
    p = kb.kvs_params_t()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = 1, 32, 8, 128
    p.window, p.sink, p.recent, p.causal = 32, 32, 32, 1
    p.softmax_scale, p.round_frac, p.score_mode, p.first_round = 128 ** -0.5, 0.5, 0, 0
    p.k_stride_b = p.v_stride_b = 8 * 4096 * 128
    p.k_stride_h = p.v_stride_h = 4096 * 128
    p.k_stride_t = p.v_stride_t = 128
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "kvs.h")).read()
    declared = set(re.findall(r"\b(kvs_[a-z_]+)\s*\(", header))
    declared.discard("kvs_workspace_size()")
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in kvs.h but not exported"
    assert set(kb.EXPORTS) == declared
    assert lib.kvs_version() >= 100


@pytest.mark.parametrize("n,budget,W,frac,first", [
    (4096, 1024, 32, 0.5, 0), (32768, 2048, 64, 0.5, 0), (16384, 1024, 32, 0.5, 1),
    (131072, 4096, 128, 0.5, 0), (2560, 2048, 32, 0.5, 0), (51451, 6431, 32, 0.5, 0),
    (1000, 999, 32, 0.01, 0), (5000, 700, 32, 0.37, 3), (300, 300, 32, 0.5, 0), (10, 300, 32, 0.5, 0),
])
def test_round_plan_matches_oracle(lib, n, budget, W, frac, first):
    p = _params(window=W, recent=W, round_frac=frac, first_round=first)
    got = kb.kvs_round_plan(p, n, budget)
    want = oc.full_plan(n, budget, 32, W, float(ctypes.c_float(frac).value), first)
    assert got == [tuple(int(x) for x in row) for row in want]


def test_round_plan_unreachable(lib):
    p = _params()
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_round_plan(p, 200, 40)        # sink + recent = 64 > budget
    assert e.value.code == 4


@pytest.mark.parametrize("field,value,code", [
    ("head_dim", 64, 2), ("n_q_heads", 30, 1), ("window", 0, 1), ("round_frac", 0.0, 1),
    ("round_frac", 1.5, 1), ("recent", 8, 1), ("score_mode", 7, 1), ("window", 512, 2),
    ("softmax_scale", 0.0, 1), ("first_round", -1, 1), ("batch", 0, 1),
])
def test_parameter_errors(lib, field, value, code):
    p = _params(**{field: value})
    if field == "window":
        p.recent = max(p.recent, value)
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_workspace_size(p, 4096)
    assert e.value.code == code
    assert kb.lib().kvs_last_error_string() != b""


def test_workspace_size_grows_with_length(lib):
    p = _params()
    a, b = kb.kvs_workspace_size(p, 4096), kb.kvs_workspace_size(p, 65536)
    assert 0 < a < b
    assert kb.kvs_workspace_size(p, 4096, 32) >= a
    with pytest.raises(kb.KvsError):
        kb.kvs_workspace_size(p, 0)
    with pytest.raises(kb.KvsError):
        kb.kvs_workspace_size(p, 4096, 1000)     # group * n_new > 1024


def test_null_pointers_are_rejected_before_any_cuda_call(lib):
    p = _params()
    one = (ctypes.c_int32 * 1)(4096)
    rc = lib.kvs_merge_layer(ctypes.byref(p), None, None, None, None, one, one, 4096, one, None,
                             ctypes.c_size_t(0), None, None)
    assert rc == 1
    rc = lib.kvs_decode_attn(ctypes.byref(p), None, 0, None, None, None, one, 4096, None, None, None,
                             ctypes.c_size_t(0), None, None)
    assert rc == 1


def test_append_and_merge_rejects_bad_arguments_before_any_cuda_call(lib):
    p = _params()
    one, zero = (ctypes.c_int32 * 1)(4096), (ctypes.c_int32 * 1)(0)
    args = lambda chunk_len, cur: (ctypes.byref(p), None, None, None, None, None, chunk_len, None, cur, one, 4096,
                                   one, None, ctypes.c_size_t(0), None, None)
    assert lib.kvs_append_and_merge(*args(-1, zero)) == 1          # negative chunk length
    assert lib.kvs_append_and_merge(*args(16, one)) == 1           # NULL chunk / no room behind 4096 slots
    assert lib.kvs_append_and_merge(*args(0, None)) == 1           # NULL cur_len
    assert b"" != lib.kvs_last_error_string()


def test_variant_entry_points_reject_bad_arguments_before_any_cuda_call(lib):
    """Exact-weight, per-head and similarity entry points: host-detectable errors come back as codes
    with nothing enqueued (all pointers here are NULL or host dummies, so a launch would fault)."""
    p = _params()
    one = (ctypes.c_int32 * 1)(4096)
    # weight_mode must be 1 or 2; e_win must not be NULL
    args = lambda mode: (ctypes.byref(p), None, None, None, None, None, mode, one, one, 4096, one, None,
                         ctypes.c_size_t(0), None, None)
    assert lib.kvs_merge_layer_exact(*args(0)) == 1
    assert lib.kvs_merge_layer_exact(*args(3)) == 1
    assert lib.kvs_merge_layer_exact(*args(1)) == 1          # NULL caches
    # per-head lengths need heads that tile the sequence stride
    bad = _params(batch=2, k_stride_b=9 * 4096 * 128)
    out = ctypes.c_size_t(0)
    assert lib.kvs_workspace_size_per_head(ctypes.byref(bad), 4096, 0, ctypes.byref(out)) == 2
    good = _params(batch=2)
    assert lib.kvs_workspace_size_per_head(ctypes.byref(good), 4096, 0, ctypes.byref(out)) == 0
    whole = kb.kvs_workspace_size(good, 4096)
    assert out.value > 0 and out.value != whole               # sized for 16 one-head sequences
    # similarity: sizes, strides, alignment
    x = ctypes.c_void_p(0x1000)
    f = lib.kvs_adjacent_cosine
    assert f(None, 1, 8, 4096, 8 * 4096 * 128, 4096 * 128, 128, one, x, None) == 1
    assert f(x, 0, 8, 4096, 8 * 4096 * 128, 4096 * 128, 128, one, x, None) == 1
    assert f(x, 1, 8, 4096, 8 * 4096 * 128, 4096 * 128, 64, one, x, None) == 1       # row stride < 128
    assert f(x, 1, 8, 4096, 8 * 4096 * 128, 4096 * 128 + 4, 128, one, x, None) == 1  # stride not a multiple of 8
    assert f(ctypes.c_void_p(0x1004), 1, 8, 4096, 8 * 4096 * 128, 4096 * 128, 128, one, x, None) == 1
    big = (ctypes.c_int32 * 1)(5000)
    assert f(x, 1, 8, 4096, 8 * 4096 * 128, 4096 * 128, 128, big, x, None) == 1      # seq_len > n_max
    # the wait hook takes three bits
    assert lib.kvs_debug_set_wait(0, 8) == 1
    assert lib.kvs_debug_set_wait(0, 0) == 0
    # the probe wants positive sizes
    assert lib.kvs_probe_sfu(0, 10, x, None, None) == 1
    pm = lib.kvs_probe_mma
    assert pm(1, 48, 0, 64, x, None) == 1           # a column count the products do not come in
    assert pm(1, 64, 0, 12, x, None) == 1           # not a multiple of 8
    assert pm(0, 64, 0, 64, x, None) == 1
    assert pm(1, 64, 0, 64, None, None) == 1
