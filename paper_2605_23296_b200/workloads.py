"""Seeded synthetic workloads for parallel context compaction attention.

This module only *draws inputs*: block lengths, a free-page list, and bf16
Q/K/V values.  It contains none of the attention or planning arithmetic, so
both the CPU oracle's tests and the CUDA path's tests can draw the same bits
from it without sharing any code of the method.

The shapes mirror the paper's setting (Section 4, "Snapshot & partition"):
an accumulated history of roughly 100k tokens is cut into N contiguous blocks
and every block is summarised by its own sequence.  Only token *counts* reach
attention, so the text of the paper's benchmarks is replaced by N(0,1) values.

All values are generated in fp32 with ``numpy.random.Generator(PCG64(seed))``
and rounded to bf16 (round-to-nearest-even); tensors are returned as
``uint16`` arrays holding the bf16 bit patterns.  Draw order is fixed:
block lengths, page permutation, Q, K, V, outlier positions, decode q/k/v.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

PAGE_SIZE = 16


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest-even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    """One synthetic compaction event: B history blocks, T summary tokens each."""

    name: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_lens: np.ndarray           # int32 [B]
    decode_steps: int                # T
    seed: int
    page_size: int = PAGE_SIZE
    permute_pages: bool = False
    outlier_scale: float = 0.0       # 0 = no outlier key
    spare_pages: int = 3             # pages in the pool beyond what the plan needs
    # filled by materialise()
    free_pages: Optional[np.ndarray] = None   # int32 [num_pages]
    q: Optional[np.ndarray] = None            # uint16 [tokens, Hq, d]
    k: Optional[np.ndarray] = None            # uint16 [tokens, Hkv, d]
    v: Optional[np.ndarray] = None
    outlier_pos: Optional[np.ndarray] = None  # int64 [B] position inside each block
    stop_lens: Optional[np.ndarray] = None    # int32 [B] tokens each sequence decodes before it stops (None: all T)
    q_dec: Optional[np.ndarray] = None        # uint16 [T, B, Hq, d]
    k_dec: Optional[np.ndarray] = None        # uint16 [T, B, Hkv, d]
    v_dec: Optional[np.ndarray] = None
    _rng: Optional[np.random.Generator] = field(default=None, repr=False)

    @property
    def num_blocks(self) -> int:
        return int(self.block_lens.shape[0])

    @property
    def total_tokens(self) -> int:
        return int(self.block_lens.astype(np.int64).sum())

    @property
    def scale(self) -> float:
        return float(1.0 / np.sqrt(np.float64(self.head_dim)))

    @property
    def pages_needed(self) -> int:
        per = (self.block_lens.astype(np.int64) + self.decode_steps + self.page_size - 1) // self.page_size
        return int(per.sum())

    @property
    def num_pages(self) -> int:
        return self.pages_needed + self.spare_pages

    def materialise(self, with_decode: bool = True) -> "Workload":
        """Draw the free list and all tensors (idempotent)."""
        if self.q is not None:
            return self
        rng = self._rng
        n_pages = self.num_pages
        if self.permute_pages:
            self.free_pages = rng.permutation(n_pages).astype(np.int32)
        else:
            self.free_pages = np.arange(n_pages, dtype=np.int32)
        tok, hq, hkv, d = self.total_tokens, self.num_q_heads, self.num_kv_heads, self.head_dim
        self.q = f32_to_bf16_bits(rng.standard_normal((tok, hq, d), dtype=np.float32))
        kf = rng.standard_normal((tok, hkv, d), dtype=np.float32)
        self.v = f32_to_bf16_bits(rng.standard_normal((tok, hkv, d), dtype=np.float32))
        if self.outlier_scale:
            # one key per block, all kv heads, scaled before the bf16 rounding
            self.outlier_pos = np.array(
                [int(rng.integers(0, int(L))) for L in self.block_lens], dtype=np.int64)
            starts = np.concatenate([[0], np.cumsum(self.block_lens.astype(np.int64))])[:-1]
            for s, p in zip(starts, self.outlier_pos):
                kf[s + p] *= np.float32(self.outlier_scale)
        self.k = f32_to_bf16_bits(kf)
        del kf
        if with_decode and self.decode_steps > 0:
            T, B = self.decode_steps, self.num_blocks
            self.q_dec = f32_to_bf16_bits(rng.standard_normal((T, B, hq, d), dtype=np.float32))
            self.k_dec = f32_to_bf16_bits(rng.standard_normal((T, B, hkv, d), dtype=np.float32))
            self.v_dec = f32_to_bf16_bits(rng.standard_normal((T, B, hkv, d), dtype=np.float32))
        return self


def _mk(name, hq, hkv, d, lens, T, seed, rng, **kw) -> Workload:
    return Workload(name=name, num_q_heads=hq, num_kv_heads=hkv, head_dim=d,
                    block_lens=np.asarray(lens, dtype=np.int32), decode_steps=T,
                    seed=seed, _rng=rng, **kw)


def tiny(seed: int = 0) -> Workload:
    """4 blocks {96,160,224,288}, GQA 4:1, d=64, 16 decode steps (parity case)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return _mk("tiny", 4, 1, 64, [96, 160, 224, 288], 16, seed, rng)


def dense8b(seed: int = 1, num_blocks: int = 8, block_len: int = 4096, steps: int = 256) -> Workload:
    """8B-class dense shape: 32q/8kv, d=128, 8 x 4096, one x8 outlier key per block."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return _mk("dense8b", 32, 8, 128, [block_len] * num_blocks, steps, seed, rng, outlier_scale=8.0)


def ragged(seed: int = 2, num_blocks: int = 32, lo: int = 1024, hi: int = 8192, steps: int = 512) -> Workload:
    """Ragged history: lengths uniform in [lo, hi], pages permuted in the pool."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(lo, hi + 1, size=num_blocks).astype(np.int32)
    return _mk("ragged", 32, 8, 128, lens, steps, seed, rng, permute_pages=True)


def moe120b(seed: int = 3, num_blocks: int = 16, block_len: int = 8192, steps: int = 512) -> Workload:
    """120B-class MoE attention shape: 64q/8kv, d=64, 16 x 8192."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return _mk("moe120b", 64, 8, 64, [block_len] * num_blocks, steps, seed, rng)


def split_sweep(num_blocks: int, seed: int = 4, history: int = 131072, steps: int = 256) -> Workload:
    """Fixed history cut into `num_blocks` equal blocks (1 = sequential compaction)."""
    assert history % num_blocks == 0
    rng = np.random.Generator(np.random.PCG64(seed))
    return _mk(f"split{num_blocks}", 32, 8, 128, [history // num_blocks] * num_blocks, steps, seed, rng)


def locomo_like(seed: int = 6, num_docs: int = 32, questions: int = 6, lo: int = 512, hi: int = 1024,
                steps: int = 256, min_stop: int = 32) -> Workload:
    """Many short sequences (the paper's second benchmark feeds documents of about 0.7k tokens with six
    questions each): num_docs x questions sequences of lo..hi tokens, 32q/8kv, d=128, whose summaries
    stop at different lengths.  `stop_lens[b]` (drawn last) is the number of tokens sequence b decodes."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n = num_docs * questions
    lens = rng.integers(lo, hi + 1, size=n).astype(np.int32)
    w = _mk("locomo_like", 32, 8, 128, lens, steps, seed, rng, permute_pages=True)
    w.stop_lens = np.random.Generator(np.random.PCG64(seed + 7919)).integers(min(min_stop, steps), steps + 1, size=n).astype(np.int32)
    return w


def custom(lens, hq, hkv, d, steps, seed=7, permute_pages=True, outlier_scale=0.0) -> Workload:
    """Arbitrary small shapes for edge-case tests."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return _mk("custom", hq, hkv, d, lens, steps, seed, rng,
               permute_pages=permute_pages, outlier_scale=outlier_scale)


def split(seed: int = 4, num_blocks: int = 8, steps: int = 256) -> Workload:
    """One point of the split sweep, addressable by name (block count as a keyword)."""
    return split_sweep(num_blocks, seed=seed, steps=steps)


@dataclass
class PrefixWorkload:
    """Inputs for the paper's prefix-aware target-at-end layout (Section 4).

    A history of `num_workers` blocks of `block_len` tokens is already cached (k_hist/v_hist, in
    `shared_pages` of the pool).  Worker w re-reads blocks 0..w-1 from that cache (prefix_lens[w] =
    w * block_len tokens) and runs its own tokens, block w wrapped in `marker_tokens` marker tokens:
    `own` holds those per-worker tokens (block_lens = block_len + marker_tokens each), their
    queries, the free pages for them and the decode-step inputs.  Page ids: the shared pages are
    0 .. hist_pages-1 (permuted together with the free pages when `own.permute_pages`)."""

    own: Workload
    block_len: int
    marker_tokens: int
    prefix_lens: np.ndarray                   # int32 [W]
    shared_pages: Optional[np.ndarray] = None  # int32 [hist_tokens / P]
    k_hist: Optional[np.ndarray] = None        # uint16 [hist_tokens, Hkv, d]
    v_hist: Optional[np.ndarray] = None

    @property
    def hist_tokens(self) -> int:
        return int(self.prefix_lens.max())

    @property
    def num_pages(self) -> int:
        return self.hist_tokens // self.own.page_size + self.own.num_pages

    def materialise(self, with_decode: bool = True) -> "PrefixWorkload":
        if self.k_hist is not None:
            return self
        o = self.own.materialise(with_decode)
        rng = o._rng
        hkv, d = o.num_kv_heads, o.head_dim
        self.k_hist = f32_to_bf16_bits(rng.standard_normal((self.hist_tokens, hkv, d), dtype=np.float32))
        self.v_hist = f32_to_bf16_bits(rng.standard_normal((self.hist_tokens, hkv, d), dtype=np.float32))
        n_shared = self.hist_tokens // o.page_size
        ids = rng.permutation(self.num_pages).astype(np.int32) if o.permute_pages else np.arange(self.num_pages, dtype=np.int32)
        self.shared_pages = ids[:n_shared].copy()
        o.free_pages = ids[n_shared:].copy()
        return self


def prefix_aware(num_workers: int, block_len: int, hq: int, hkv: int, d: int, steps: int, seed: int = 11,
                 marker_tokens: int = 16, permute_pages: bool = True, own_len: int = 0,
                 own_lens: Optional[Sequence[int]] = None) -> PrefixWorkload:
    """`num_workers` workers over a history of blocks of `block_len` tokens (a multiple of 128);
    `own_len` > 0 replaces the workers' own length (block + markers), `own_lens` gives every worker
    its own, for edge cases."""
    assert block_len % 128 == 0 and num_workers >= 1
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = list(own_lens) if own_lens is not None else [own_len or block_len + marker_tokens] * num_workers
    assert len(lens) == num_workers
    own = _mk(f"prefix{num_workers}x{block_len}", hq, hkv, d, lens, steps, seed, rng, permute_pages=permute_pages)
    pre = np.arange(num_workers, dtype=np.int32) * np.int32(block_len)
    return PrefixWorkload(own=own, block_len=block_len, marker_tokens=marker_tokens, prefix_lens=pre)


CONFIGS = {
    "tiny": tiny,
    "dense8b": dense8b,
    "ragged": ragged,
    "moe120b": moe120b,
    "split": split,
    "locomo_like": locomo_like,
}
