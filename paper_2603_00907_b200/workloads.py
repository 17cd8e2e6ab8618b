"""Seeded synthetic inputs for the KV-merge pass.

This module holds no arithmetic of the merge method itself.  It only draws the
bf16 keys, value sums, window queries and decode queries that stand in for the
long-context workloads the paper evaluates (Llama-3.1-8B-, Qwen2.5-7B- and
Llama-3-70B-shaped caches): adjacent keys are homogeneous (an AR(1) drift along
the token axis plus a constant offset on a few outlier channels), values are
i.i.d. and therefore heterogeneous, queries are i.i.d. standard normal.

Everything is generated on the CPU with numpy, rounded to bf16
(round-to-nearest-even) and returned as uint16 bit patterns so that every
consumer sees exactly the same bits.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
from scipy.signal import lfilter

HEAD_DIM = 128


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and generator parameters of one benchmark configuration."""
    name: str
    config_id: int
    layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    window: int
    seq_lens: tuple            # per sequence
    budgets: tuple             # per sequence
    ar_coef: Optional[float]   # None: drawn per layer from U[ar_lo, ar_hi]
    ar_lo: float = 0.8
    ar_hi: float = 0.95
    noise_literal: Optional[float] = None   # fixed innovation std; None -> sqrt(1-a^2)
    n_outlier: int = 8
    outlier_std: float = 2.0
    n_decode: int = 0          # new query tokens per sequence for the decode check
    sink: int = 32
    round_frac: float = 0.5

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_max(self) -> int:
        return int(max(self.seq_lens))

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _ragged_lengths(seed: int, batch: int, lo: int, hi: int) -> tuple:
    rng = np.random.default_rng(seed)
    return tuple(int(v) for v in rng.integers(lo, hi + 1, size=batch))


def config(config_id: int) -> Workload:
    """The five benchmark configurations."""
    if config_id == 0:
        return Workload("llama31_8b_1layer_ctx4k", 0, 1, 1, 32, 8, 32, (4096,), (1024,),
                        ar_coef=0.9, noise_literal=0.44, n_outlier=8, outlier_std=2.0)
    if config_id == 1:
        return Workload("llama31_8b_32layer_ctx32k", 1, 32, 1, 32, 8, 64, (32768,), (2048,),
                        ar_coef=None, n_outlier=8, outlier_std=2.0)
    if config_id == 2:
        return Workload("qwen25_7b_28layer_b4_ctx16k", 2, 28, 4, 28, 4, 32, (16384,) * 4,
                        (1024,) * 4, ar_coef=0.9, noise_literal=0.44, n_outlier=4,
                        outlier_std=2.0)
    if config_id == 3:
        lens = _ragged_lengths(3000, 8, 4096, 65536)
        return Workload("llama31_8b_ragged_b8", 3, 1, 8, 32, 8, 32, lens,
                        tuple(n // 8 for n in lens), ar_coef=0.9, noise_literal=0.44,
                        n_outlier=8, outlier_std=2.0, n_decode=32)
    if config_id == 4:
        return Workload("llama3_70b_1layer_ctx128k", 4, 1, 1, 64, 8, 128, (131072,), (4096,),
                        ar_coef=0.92, n_outlier=8, outlier_std=3.0, n_decode=32)
    raise ValueError(f"unknown config {config_id}")


def layer_ar_coef(w: Workload, layer: int) -> float:
    if w.ar_coef is not None:
        return float(w.ar_coef)
    rng = np.random.default_rng(1000 * w.config_id + 7919)
    coefs = rng.uniform(w.ar_lo, w.ar_hi, size=w.layers)
    return float(coefs[layer])


def _ar1(rng: np.random.Generator, n: int, width: int, a: float, sigma: float) -> np.ndarray:
    """x_0 ~ N(0,1); x_t = a x_{t-1} + sigma eps_t along the token axis.  Returns [n, width]."""
    eps = rng.standard_normal((width, n), dtype=np.float32)      # channel-major: filter rows
    eps[:, 1:] *= np.float32(sigma)
    # y_t = a y_{t-1} + u_t with u_0 = x_0 and zero initial state
    y = lfilter([1.0], [1.0, -a], eps.astype(np.float64), axis=1).astype(np.float32)
    return np.ascontiguousarray(y.T)


def make_layer(w: Workload, layer: int = 0, seq_offset: int = 0) -> Dict[str, np.ndarray]:
    """Inputs of one decoder layer.

    Returns uint16 (bf16 bits) arrays K, V [B,Hkv,Nmax,128], q_win [B,Hq,W,128],
    q_new [B,Hq,T,128] (T = n_decode, may be 0), int32 counts [B,Hkv,Nmax] (all 1),
    and int32 seq_len / budget [B].  Rows at or beyond seq_len[b] are zero.
    `seq_offset` shifts the per-sequence seeds (another data-parallel rank's batch).
    """
    B, Hq, Hkv, W, d = w.batch, w.n_q_heads, w.n_kv_heads, w.window, HEAD_DIM
    nmax = w.n_max
    a = layer_ar_coef(w, layer)
    sigma = w.noise_literal if w.noise_literal is not None else float(np.sqrt(1.0 - a * a))
    K = np.zeros((B, Hkv, nmax, d), dtype=np.uint16)
    V = np.zeros((B, Hkv, nmax, d), dtype=np.uint16)
    q_win = np.zeros((B, Hq, W, d), dtype=np.uint16)
    q_new = np.zeros((B, Hq, w.n_decode, d), dtype=np.uint16)
    for b in range(B):
        base = 1000 * w.config_id + 10 * layer + b + 100000 * seq_offset
        n = int(w.seq_lens[b])
        rk = np.random.default_rng([base, 1])
        rv = np.random.default_rng([base, 2])
        rq = np.random.default_rng([base, 3])
        ro = np.random.default_rng([1000 * w.config_id + 10 * layer, 4])
        rd = np.random.default_rng([base, 5])
        keys = _ar1(rk, n, Hkv * d, a, sigma).reshape(n, Hkv, d)
        for h in range(Hkv):
            ch = ro.choice(d, size=w.n_outlier, replace=False)
            off = (w.outlier_std * ro.standard_normal(w.n_outlier)).astype(np.float32)
            keys[:, h, ch] += off[None, :]
        K[b, :, :n, :] = f32_to_bf16_bits(keys).transpose(1, 0, 2)
        vals = rv.standard_normal((n, Hkv, d), dtype=np.float32)
        V[b, :, :n, :] = f32_to_bf16_bits(vals).transpose(1, 0, 2)
        q_win[b] = f32_to_bf16_bits(rq.standard_normal((Hq, W, d), dtype=np.float32))
        if w.n_decode:
            q_new[b] = f32_to_bf16_bits(rd.standard_normal((Hq, w.n_decode, d), dtype=np.float32))
    counts = np.zeros((B, Hkv, nmax), dtype=np.int32)
    for b in range(B):
        counts[b, :, : int(w.seq_lens[b])] = 1
    return {
        "K": K, "V": V, "counts": counts, "q_win": q_win, "q_new": q_new,
        "seq_len": np.asarray(w.seq_lens, dtype=np.int32),
        "budget": np.asarray(w.budgets, dtype=np.int32),
    }


def small_case(seed: int, batch: int = 1, n_q_heads: int = 8, n_kv_heads: int = 2,
               window: int = 8, seq_lens=(300,), budgets=(100,), n_decode: int = 0,
               ar_coef: float = 0.9, n_outlier: int = 4) -> Workload:
    """A reduced workload with the same structure, for parity tests."""
    return Workload(f"small_{seed}", 100 + seed, 1, batch, n_q_heads, n_kv_heads, window,
                    tuple(seq_lens), tuple(budgets), ar_coef=ar_coef, noise_literal=None,
                    n_outlier=n_outlier, outlier_std=2.0, n_decode=n_decode)


def make_layers_parallel(w: Workload, layers, processes: Optional[int] = None, seq_offset: int = 0) -> List[Dict[str, np.ndarray]]:
    """make_layer for several layers on a process pool (generation is the slow part of a
    benchmark set-up; results are identical to calling make_layer one by one)."""
    import multiprocessing as mp
    import os
    layers = list(layers)
    procs = processes or min(len(layers), max(1, (os.cpu_count() or 2) - 1), 16)
    if procs <= 1 or len(layers) <= 1:
        return [make_layer(w, l, seq_offset) for l in layers]
    with mp.get_context("fork").Pool(procs) as pool:
        return pool.starmap(make_layer, [(w, l, seq_offset) for l in layers])
