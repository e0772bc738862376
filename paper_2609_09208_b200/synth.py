"""Seeded synthetic inputs with the shapes and value structure of the paper's workloads.

This module only draws random numbers and shapes them; it contains none of the method's
arithmetic (no quantiser, no score, no softmax), so that the CPU oracle and the CUDA
library can both be fed from it without sharing any code of the method itself.

The paper measured on post-RoPE tensors of a 1.1 B-parameter Llama decoder (22 layers,
32 query heads, 4 KV heads, head_dim 64).  Neither those weights nor the text corpus are
available, so the tensors are stood in for by seeded Gaussians; where a workload asks for
"outlier" keys, each (KV head, channel) gets one log-normal(0, 1) multiplier, which is the
per-channel outlier structure a Hadamard rotation is meant to flatten.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

LLAMA_1B_LAYERS = 22  # decoder layers of the paper's model (section IV)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def gaussian_fp16(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float32).astype(np.float16)


def outlier_keys_fp16(rng: np.random.Generator, n_tokens: int, n_kv_heads: int, d: int) -> np.ndarray:
    """N(0,1) keys times one log-normal(0,1) multiplier per (KV head, channel)."""
    chan = np.exp(rng.standard_normal((1, n_kv_heads, d), dtype=np.float32))
    k = rng.standard_normal((n_tokens, n_kv_heads, d), dtype=np.float32) * chan
    return k.astype(np.float16)


def ragged_lens(rng: np.random.Generator, batch: int, lo: int, hi: int) -> np.ndarray:
    return rng.integers(lo, hi + 1, size=batch).astype(np.int64)


@dataclass
class Case:
    """One decode step's inputs: Q [B,Hq,d]; K,V [sum T_b,Hkv,d] (float16); cu_lens int64 [B+1]."""
    name: str
    Q: np.ndarray
    K: np.ndarray
    V: np.ndarray
    cu_lens: np.ndarray
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    code_k: int                   # mantissa bits: 0 (PoT-4), 1, 2, 4
    nibble: bool = False          # PoT-4 stored two codes per byte
    hadamard: bool = False
    seed: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def lens(self) -> np.ndarray:
        return np.diff(self.cu_lens)

    @property
    def batch(self) -> int:
        return len(self.cu_lens) - 1

    @property
    def n_keys(self) -> int:
        """Cached (token, KV head) vectors: the unit of the keys/s metric."""
        return int(self.cu_lens[-1]) * self.n_kv_heads


def make_case(name: str, lens, n_q_heads: int, n_kv_heads: int, d: int, code_k: int, *,
              outliers: bool = False, nibble: bool = False, hadamard: bool = False,
              seed: int = 0) -> Case:
    rng = _rng(seed)
    lens = np.asarray(lens, dtype=np.int64)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(cu[-1])
    Q = gaussian_fp16(rng, (len(lens), n_q_heads, d))
    K = outlier_keys_fp16(rng, total, n_kv_heads, d) if outliers else gaussian_fp16(rng, (total, n_kv_heads, d))
    V = gaussian_fp16(rng, (total, n_kv_heads, d))
    return Case(name, Q, K, V, cu, n_q_heads, n_kv_heads, d, code_k, nibble=nibble, hadamard=hadamard,
                seed=seed)


# The five workloads.  Each function returns the full-size case unless `scale_T` shrinks it
# (tests use smaller T where the CPU oracle has to run the whole thing element by element).

def config1(seed: int = 0) -> Case:
    """Single head, d=64, one query, T=1024, N(0,1) everything, PoT-4."""
    return make_case("cfg1_single_head_T1024_pot4", [1024], 1, 1, 64, 0, seed=seed)


def config2(seed: int = 2000, T: int = 4096) -> Case:
    """Llama-1.1B-shaped step: 32/4 heads, d=64, T=4096, outlier K, PoT-M1 byte code."""
    return make_case("cfg2_llama1b_T%d_potm1" % T, [T], 32, 4, 64, 1, outliers=True, seed=seed)


def config3(code_k: int = 4, *, hadamard: bool = False, nibble: bool = False, outliers: bool = False,
            T: int = 32768, batch: int = 1, seed: int = 3000) -> Case:
    """32/4 heads, d=64, T=32768; PoT-4 / PoT-M4, with or without rotation."""
    name = "cfg3_T%d_B%d_k%d%s%s%s" % (T, batch, code_k, "_had" if hadamard else "",
                                         "_nib" if nibble else "", "_out" if outliers else "")
    return make_case(name, [T] * batch, 32, 4, 64, code_k, outliers=outliers, nibble=nibble,
                     hadamard=hadamard, seed=seed + code_k)


def config4(seed: int = 4000, batch: int = 16, lo: int = 2048, hi: int = 16384) -> Case:
    """Batched ragged decode: B=16, lengths uniform in [2048, 16384], PoT-M2, outlier K."""
    lens = ragged_lens(_rng(seed + 1), batch, lo, hi)
    return make_case("cfg4_ragged_B%d_potm2" % batch, lens, 32, 4, 64, 2, outliers=True, seed=seed)


def config5(T: int, batch: int, code_k: int, seed: int = 5000) -> Case:
    """Long-context sweep cell: 32/8 heads, d=128, outlier K."""
    return make_case("cfg5_T%d_B%d_k%d" % (T, batch, code_k), [T] * batch, 32, 8, 128, code_k,
                     outliers=True, seed=seed + code_k)


def page_permutation(n_pages: int, seed: int) -> np.ndarray:
    """A random assignment of logical pages to physical pool slots (paged KV cache)."""
    return _rng(seed).permutation(n_pages).astype(np.int32)
