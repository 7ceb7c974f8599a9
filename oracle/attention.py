"""fp64 attention by the plain definition.  TEST INFRASTRUCTURE ONLY.

Thin ctypes layer over ``attn_oracle.c`` plus the pieces that are simpler to
state in numpy: the contiguous-KV decode state, the expected contents of a
paged pool, and the log-sum-exp merge of split partial results.

The paper (Section 4) fixes the block structure: N independent blocks, one
summary sequence per block, summaries concatenated in block order.  Attention
itself is the textbook causal softmax attention with grouped-query heads
(query head h reads kv head h div G).  A decode step appends the new token's
key/value first and then attends over all cached keys, the new one included,
so step t of block b equals the last row of a causal prefill over the
(L_b + t + 1)-token sequence.

The paper's own layout (Section 4, "Prefix-aware target-at-end layout") is
covered by ``prefill_prefix_aware`` / ``PrefixDecodeState``: the prompt of
worker w is the history up to its block followed by its own (target) tokens, so
a target token attends causally over that whole prompt; it is written here as
exactly that, the plain causal attention over the concatenated prompt.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

from . import _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        i64p = ctypes.POINTER(ctypes.c_int64)
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.oracle_prefill.argtypes = [u16p, u16p, u16p, i32p, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int, ctypes.c_int, ctypes.c_double, i64p,
                                       ctypes.c_int64, f64p, ctypes.c_int]
        lib.oracle_prefill.restype = ctypes.c_int
        lib.oracle_attend_token.argtypes = [u16p, u16p, u16p, ctypes.c_int64, ctypes.c_int,
                                            ctypes.c_int, ctypes.c_int, ctypes.c_double, f64p, f64p]
        lib.oracle_attend_token.restype = ctypes.c_int
        _lib = lib
    return _lib


def host_threads() -> int:
    """Cores this process may run on (what the threaded prefill will use)."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _u16(a):
    a = np.ascontiguousarray(a, dtype=np.uint16)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def prefill(q: np.ndarray, k: np.ndarray, v: np.ndarray, cu_seqlens: Sequence[int],
            scale: float, rows: Optional[Sequence[int]] = None,
            threads: Optional[int] = None) -> np.ndarray:
    """Causal attention inside every block of a packed ragged batch.

    q [tokens,Hq,d], k/v [tokens,Hkv,d] as bf16 bits.  Returns float64
    [tokens,Hq,d], or [len(rows),Hq,d] when `rows` (global token ids) is given.
    """
    lib = _load()
    tokens, Hq, d = q.shape
    Hkv = k.shape[1]
    assert k.shape == (tokens, Hkv, d) and v.shape == k.shape
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    assert int(cu[-1]) == tokens and cu[0] == 0
    B = cu.shape[0] - 1
    qa, qp = _u16(q)
    ka, kp = _u16(k)
    va, vp = _u16(v)
    if rows is None:
        rows_p, n_rows = None, tokens
    else:
        rows_a = np.ascontiguousarray(rows, dtype=np.int64)
        assert rows_a.ndim == 1 and (rows_a >= 0).all() and (rows_a < tokens).all()
        rows_p, n_rows = rows_a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), rows_a.shape[0]
    out = np.empty((n_rows, Hq, d), dtype=np.float64)
    rc = lib.oracle_prefill(qp, kp, vp, cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), B, Hq,
                            Hkv, d, float(scale), rows_p, n_rows,
                            out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                            int(threads or host_threads()))
    if rc != 0:
        raise ValueError("oracle_prefill: bad arguments")
    return out


def attend_token(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float,
                 return_weights: bool = False):
    """One query token q [Hq,d] over all n keys of k/v [n,Hkv,d] (bf16 bits)."""
    lib = _load()
    Hq, d = q.shape
    n, Hkv, _ = k.shape
    qa, qp = _u16(q)
    ka, kp = _u16(k)
    va, vp = _u16(v)
    out = np.empty((Hq, d), dtype=np.float64)
    p = np.empty((Hq, n), dtype=np.float64) if return_weights else None
    rc = lib.oracle_attend_token(qp, kp, vp, n, Hq, Hkv, d, float(scale),
                                 out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                 p.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if return_weights else None)
    if rc != 0:
        raise ValueError("oracle_attend_token: bad arguments")
    return (out, p) if return_weights else out


def prefill_chunk(q: np.ndarray, k: np.ndarray, v: np.ndarray, cu_seqlens: Sequence[int], scale: float,
                  block: int, first_row: int, n_rows: int) -> np.ndarray:
    """One chunk of a chunked prefill (Section 4.2: the engine prefills long prompts in chunks).

    When rows [first_row, first_row + n_rows) of `block` are prefilled, the block's later tokens do
    not exist yet: the chunk attends, causally, over the block's tokens [0, first_row + n_rows) and
    nothing else.  Written as exactly that: the block is cut off behind the chunk and the plain
    causal attention is evaluated for the chunk's rows.  Returns float64 [n_rows, Hq, d].
    """
    lo = int(cu_seqlens[block])
    end = first_row + n_rows
    assert 0 <= first_row and n_rows >= 1 and lo + end <= int(cu_seqlens[block + 1])
    return prefill(q[lo:lo + end], k[lo:lo + end], v[lo:lo + end], [0, end], scale,
                   rows=np.arange(first_row, end, dtype=np.int64))


class DecodeState:
    """Per-block contiguous K/V (independent of any page table).

    `append` adds one token per block; `decode` evaluates the new query token
    of every block over that block's whole cache (new token included).
    """

    def __init__(self, k: np.ndarray, v: np.ndarray, cu_seqlens: Sequence[int], max_new: int):
        cu = [int(x) for x in cu_seqlens]
        self.B = len(cu) - 1
        _, self.Hkv, self.d = k.shape
        self.len = [cu[b + 1] - cu[b] for b in range(self.B)]
        self.k, self.v = [], []
        for b in range(self.B):
            cap = self.len[b] + max_new
            kb = np.zeros((cap, self.Hkv, self.d), dtype=np.uint16)
            vb = np.zeros_like(kb)
            kb[: self.len[b]] = k[cu[b]:cu[b + 1]]
            vb[: self.len[b]] = v[cu[b]:cu[b + 1]]
            self.k.append(kb)
            self.v.append(vb)

    def append(self, k_new: np.ndarray, v_new: np.ndarray, blocks: Optional[Sequence[int]] = None) -> None:
        """k_new, v_new: [B,Hkv,d] bf16 bits, one token per block (only for `blocks` when given: the
        others sit the step out)."""
        for b in (range(self.B) if blocks is None else blocks):
            self.k[b][self.len[b]] = k_new[b]
            self.v[b][self.len[b]] = v_new[b]
            self.len[b] += 1

    def decode(self, q: np.ndarray, scale: float, blocks: Optional[Sequence[int]] = None) -> np.ndarray:
        """q [B,Hq,d] bf16 bits -> float64 [B,Hq,d] (rows of unselected blocks are NaN)."""
        out = np.full((self.B,) + q.shape[1:], np.nan, dtype=np.float64)
        for b in (range(self.B) if blocks is None else blocks):
            n = self.len[b]
            out[b] = attend_token(q[b], self.k[b][:n], self.v[b][:n], scale)
        return out


def prefill_prefix_aware(q: np.ndarray, k: np.ndarray, v: np.ndarray, cu_seqlens: Sequence[int],
                         k_hist: np.ndarray, v_hist: np.ndarray, prefix_lens: Sequence[int],
                         scale: float, rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Attention of every worker's own tokens over its prompt (Section 4, "Dispatch").

    Worker w's prompt is the first prefix_lens[w] tokens of the shared history
    (k_hist/v_hist [hist_tokens,Hkv,d]) followed by its own tokens
    k/v[cu[w]:cu[w+1]] (the target block with its markers).  Row i of worker w
    sees the whole prefix and its own tokens 0..i: causal attention over the
    concatenated prompt, evaluated for the rows of the own tokens only.
    q [tokens,Hq,d] holds the own tokens' queries (the prefix needs none).
    Returns float64 [tokens,Hq,d], or [len(rows),Hq,d] for `rows` (ids into q).
    """
    cu = [int(x) for x in cu_seqlens]
    W = len(cu) - 1
    tokens, Hq, d = q.shape
    assert len(prefix_lens) == W and cu[-1] == tokens
    wanted = None if rows is None else [int(r) for r in rows]
    out = np.empty((tokens if wanted is None else len(wanted), Hq, d), dtype=np.float64)
    for w in range(W):
        n_pre, lo, hi = int(prefix_lens[w]), cu[w], cu[w + 1]
        assert 0 <= n_pre <= k_hist.shape[0]
        if wanted is None:
            local, dest = list(range(hi - lo)), list(range(lo, hi))
        else:
            sel = [(i, r - lo) for i, r in enumerate(wanted) if lo <= r < hi]
            if not sel:
                continue
            dest, local = [i for i, _ in sel], [r for _, r in sel]
        prompt_k = np.concatenate([k_hist[:n_pre], k[lo:hi]])
        prompt_v = np.concatenate([v_hist[:n_pre], v[lo:hi]])
        prompt_q = np.concatenate([np.zeros((n_pre, Hq, d), dtype=np.uint16), q[lo:hi]])
        res = prefill(prompt_q, prompt_k, prompt_v, [0, n_pre + hi - lo], scale,
                      rows=[n_pre + r for r in local])
        out[dest] = res
    return out


def prefill_chunk_prefix_aware(q: np.ndarray, k: np.ndarray, v: np.ndarray, cu_seqlens: Sequence[int],
                               k_hist: np.ndarray, v_hist: np.ndarray, prefix_lens: Sequence[int], scale: float,
                               worker: int, first_row: int, n_rows: int) -> np.ndarray:
    """One chunk of a worker's chunked prefill in the prefix-aware layout (Section 4 "Dispatch" for the prompt,
    Section 4.2 for prefix caching and chunked prefill being on together in the paper's serving engine).

    Worker w's prompt is its history prefix followed by its own tokens.  When rows [first_row, first_row + n_rows)
    of the own tokens are prefilled, the later own tokens do not exist yet: the chunk attends, causally, over the
    prefix and the own tokens [0, first_row + n_rows).  Written as that: the prompt is cut off behind the chunk and
    plain causal attention is evaluated for the chunk's rows.  Returns float64 [n_rows, Hq, d].
    """
    lo, n_pre = int(cu_seqlens[worker]), int(prefix_lens[worker])
    end = first_row + n_rows
    assert 0 <= first_row and n_rows >= 1 and lo + end <= int(cu_seqlens[worker + 1])
    Hq, d = q.shape[1], q.shape[2]
    prompt_k = np.concatenate([k_hist[:n_pre], k[lo:lo + end]])
    prompt_v = np.concatenate([v_hist[:n_pre], v[lo:lo + end]])
    prompt_q = np.concatenate([np.zeros((n_pre, Hq, d), dtype=np.uint16), q[lo:lo + end]])
    return prefill(prompt_q, prompt_k, prompt_v, [0, n_pre + end], scale,
                   rows=np.arange(n_pre + first_row, n_pre + end, dtype=np.int64))


class PrefixDecodeState(DecodeState):
    """Decode in the prefix-aware layout: worker w's cache is its prompt (history prefix, then its
    own tokens), kept contiguously per worker and extended one token per step."""

    def __init__(self, k: np.ndarray, v: np.ndarray, cu_seqlens: Sequence[int], k_hist: np.ndarray,
                 v_hist: np.ndarray, prefix_lens: Sequence[int], max_new: int):
        cu = [int(x) for x in cu_seqlens]
        ks, vs, ccu = [], [], [0]
        for w in range(len(cu) - 1):
            n_pre = int(prefix_lens[w])
            ks += [k_hist[:n_pre], k[cu[w]:cu[w + 1]]]
            vs += [v_hist[:n_pre], v[cu[w]:cu[w + 1]]]
            ccu.append(ccu[-1] + n_pre + cu[w + 1] - cu[w])
        super().__init__(np.concatenate(ks), np.concatenate(vs), ccu, max_new)


def expected_pool(slot_mapping: Sequence[int], k: np.ndarray, v: np.ndarray,
                  num_pages: int, page_size: int):
    """Pool contents after appending token i of the packed batch to slot_mapping[i].

    Pools are [num_pages, Hkv, P, d]; returns (k_pool, v_pool, written) where
    `written` [num_pages, P] marks slots that hold a token.
    """
    tokens, Hkv, d = k.shape
    k_pool = np.zeros((num_pages, Hkv, page_size, d), dtype=np.uint16)
    v_pool = np.zeros_like(k_pool)
    written = np.zeros((num_pages, page_size), dtype=bool)
    for i in range(tokens):
        page, off = divmod(int(slot_mapping[i]), page_size)
        k_pool[page, :, off, :] = k[i]
        v_pool[page, :, off, :] = v[i]
        written[page, off] = True
    return k_pool, v_pool, written


def split_partial(q_head: np.ndarray, k_head: np.ndarray, v_head: np.ndarray, scale: float):
    """(m, l, acc) of one key range: m = max score, l = sum exp(s-m), acc = sum exp(s-m) v.

    All float64; q_head [d], k_head/v_head [n,d].  An empty range gives (-inf, 0, 0).
    """
    if k_head.shape[0] == 0:
        return -np.inf, 0.0, np.zeros(v_head.shape[1], dtype=np.float64)
    s = scale * (k_head @ q_head)
    m = float(s.max())
    p = np.exp(s - m)
    return m, float(p.sum()), p @ v_head


def combine_splits(ms, ls, accs) -> np.ndarray:
    """Merge split partials: m = max m_s; l = sum l_s e^(m_s-m); O = sum acc_s e^(m_s-m) / l."""
    m = max(ms)
    l = 0.0
    o = np.zeros_like(accs[0])
    for ms_, ls_, acc in zip(ms, ls, accs):
        if ls_ == 0.0:
            continue
        w = np.exp(ms_ - m)
        l += ls_ * w
        o = o + acc * w
    return o / l
