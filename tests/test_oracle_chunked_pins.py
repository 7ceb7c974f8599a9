"""Pins of the oracle's chunked-prefill pieces (paper, Section 4.2: chunked prefill is enabled in the
serving engine; Section 6: 16k blocks are prefill-bound).  The schedule is pinned by a hand-worked
table and by what any valid schedule must satisfy; the chunk's attention by the identity that makes
chunking legitimate at all: cutting a causal prefill into chunks changes no output row."""
import os

import numpy as np
import pytest

from oracle import attention as oa
from oracle import plan as op
from paper_2605_23296_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "mixed_schedule_small.txt")


def _read_golden():
    head, steps = {}, []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if "|" not in line:
            key, *vals = line.split()
            head[key] = [int(x) for x in vals]
            continue
        _, pre, dec = [x.strip() for x in line.split("|")]
        steps.append({"prefill": [tuple(int(y) for y in x.split(":")) for x in pre.split()],
                      "decode": [int(x) for x in dec.split()]})
    return head, steps


def test_mixed_schedule_matches_the_hand_worked_table():
    head, steps = _read_golden()
    got = op.mixed_schedule(head["block_lens"], head["chunk_tokens"][0], head["max_new_tokens"][0],
                            head["decode_steps_per_chunk"][0])
    assert got == steps
    # one decode step per chunk: the same chunks and decoders without the steps in between
    lock = op.mixed_schedule(head["block_lens"], head["chunk_tokens"][0], 2, 1)
    assert lock == [{"prefill": [(0, 0, 128), (1, 0, 100), (2, 0, 50)], "decode": []},
                    {"prefill": [(0, 128, 128)], "decode": [1, 2]}, {"prefill": [(0, 256, 44)], "decode": [1, 2]},
                    {"prefill": [], "decode": [0]}, {"prefill": [], "decode": [0]}]


@pytest.mark.parametrize("lens,C,T,r", [([16384, 2048, 2048, 2048, 2048], 2048, 256, 1), ([1, 129, 128, 1000], 128, 3, 1),
                                         ([700], 256, 0, 1), ([5, 5, 5], 1024, 4, 1), ([16384, 2048, 2048], 2048, 40, 16),
                                         ([300, 100, 50], 128, 2, 3)])
def test_mixed_schedule_invariants(lens, C, T, r):
    steps = op.mixed_schedule(lens, C, T, r)
    rows_done = [0] * len(lens)
    last_chunk_step = [None] * len(lens)
    decoded = [[] for _ in lens]
    for s, st in enumerate(steps):
        assert not st["prefill"] or s % r == 0                    # a chunk starts every r steps
        for b, first, n in st["prefill"]:
            assert first == rows_done[b] and 1 <= n <= C          # chunks in order, nothing skipped or repeated
            assert n == C or first + n == lens[b]                 # only a block's last chunk is short
            rows_done[b] += n
            last_chunk_step[b] = s
        for b in st["decode"]:
            assert rows_done[b] == lens[b]                        # a block decodes only after its whole prefill ...
            assert s >= last_chunk_step[b] + r                    # ... has had its r steps
            decoded[b].append(s)
    assert rows_done == list(lens)
    for b, d in enumerate(decoded):
        n_b = -(-lens[b] // C)
        assert len(d) == T and d == list(range(n_b * r, n_b * r + T))   # T steps in a row, at once
    assert len(steps) == max(-(-L // C) for L in lens) * r + T


def test_mixed_schedule_with_one_chunk_is_prefill_then_decode():
    # a chunk at least as long as every block: step 0 prefills everything, then T plain decode steps
    steps = op.mixed_schedule([96, 160, 224], 4096, 3)
    assert steps[0] == {"prefill": [(0, 0, 96), (1, 0, 160), (2, 0, 224)], "decode": []}
    assert steps[1:] == [{"prefill": [], "decode": [0, 1, 2]}] * 3


def test_mixed_schedule_rejects_bad_input():
    for args in [([10], 0, 1), ([10], 8, -1), ([], 8, 1), ([0], 8, 1), ([10], 8, 1, 0)]:
        with pytest.raises(ValueError):
            op.mixed_schedule(*args)


def test_chunk_rows_equal_the_unchunked_prefill_rows_bitwise():
    # the identity chunked prefill rests on: a causal row never sees the tokens behind it, so
    # evaluating a chunk with the rest of the block cut off gives the very same fp64 numbers
    w = wl.custom([300, 77, 130], 4, 2, 64, steps=0, seed=5).materialise()
    cu = np.concatenate([[0], np.cumsum(w.block_lens.astype(np.int64))])
    full = oa.prefill(w.q, w.k, w.v, cu, w.scale)
    for st in op.mixed_schedule(w.block_lens.tolist(), 128, 0):
        for b, first, n in st["prefill"]:
            got = oa.prefill_chunk(w.q, w.k, w.v, cu, w.scale, b, first, n)
            assert np.array_equal(got, full[cu[b] + first: cu[b] + first + n])


def test_chunk_sees_earlier_chunks_and_not_later_tokens():
    w = wl.custom([260], 2, 1, 64, steps=0, seed=6).materialise()
    cu = [0, 260]
    base = oa.prefill_chunk(w.q, w.k, w.v, cu, w.scale, 0, 128, 128)
    k2 = w.k.copy()
    k2[256:] ^= 0x4000                      # tokens behind the chunk: no effect
    assert np.array_equal(oa.prefill_chunk(w.q, k2, w.v, cu, w.scale, 0, 128, 128), base)
    v2 = w.v.copy()
    v2[5] ^= 0x0100                         # a token of the first chunk: every row of the second one moves
    moved = oa.prefill_chunk(w.q, w.k, v2, cu, w.scale, 0, 128, 128)
    assert (np.abs(moved - base).max(axis=(1, 2)) > 0).all()


def test_chunk_first_row_of_first_chunk_is_its_own_value():
    w = wl.custom([40], 2, 2, 64, steps=0, seed=8).materialise()
    got = oa.prefill_chunk(w.q, w.k, w.v, [0, 40], w.scale, 0, 0, 16)
    assert np.array_equal(got[0], oa.bf16_bits_to_f64(w.v[0]))


def test_decode_state_lets_blocks_sit_a_step_out():
    w = wl.custom([20, 30], 2, 1, 64, steps=2, seed=9).materialise()
    cu = [0, 20, 50]
    st = oa.DecodeState(w.k, w.v, cu, 2)
    st.append(w.k_dec[0], w.v_dec[0], blocks=[1])
    assert st.len == [20, 31]
    out = st.decode(w.q_dec[0], w.scale, blocks=[1])
    want = oa.attend_token(w.q_dec[0][1], np.concatenate([w.k[20:50], w.k_dec[0][1:2]]),
                           np.concatenate([w.v[20:50], w.v_dec[0][1:2]]), w.scale)
    assert np.array_equal(out[1], want) and np.isnan(out[0]).all()


def test_prefix_aware_chunk_rows_equal_the_unchunked_prefix_aware_rows_bitwise():
    # the same identity with a cached history in front: chunking a worker's own tokens changes none of its rows
    pw = wl.prefix_aware(3, 128, 4, 2, 64, steps=0, seed=12, marker_tokens=45).materialise(with_decode=False)
    o = pw.own
    cu = np.concatenate([[0], np.cumsum(o.block_lens.astype(np.int64))])
    full = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, pw.k_hist, pw.v_hist, pw.prefix_lens, o.scale)
    for st in op.mixed_schedule(o.block_lens.tolist(), 128, 0):
        for w, first, n in st["prefill"]:
            got = oa.prefill_chunk_prefix_aware(o.q, o.k, o.v, cu, pw.k_hist, pw.v_hist, pw.prefix_lens, o.scale, w, first, n)
            assert np.array_equal(got, full[cu[w] + first: cu[w] + first + n])
    # worker 0 has no prefix: its chunks are the independent-chunks ones
    got = oa.prefill_chunk_prefix_aware(o.q, o.k, o.v, cu, pw.k_hist, pw.v_hist, pw.prefix_lens, o.scale, 0, 128, 45)
    assert np.array_equal(got, oa.prefill_chunk(o.q, o.k, o.v, cu, o.scale, 0, 128, 45))
    # a chunk of worker 2 sees the history inside its prefix and not the history beyond it
    base = oa.prefill_chunk_prefix_aware(o.q, o.k, o.v, cu, pw.k_hist, pw.v_hist, pw.prefix_lens, o.scale, 2, 128, 45)
    kh = pw.k_hist.copy()
    kh[3] ^= 0x0100
    moved = oa.prefill_chunk_prefix_aware(o.q, o.k, o.v, cu, kh, pw.v_hist, pw.prefix_lens, o.scale, 2, 128, 45)
    assert (np.abs(moved - base).max(axis=(1, 2)) > 0).all()
