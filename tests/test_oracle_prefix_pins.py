"""Pins for the oracle's prefix-aware layout (paper, Section 4, "Prefix-aware target-at-end
layout"): each check ties it to something other than itself: the already pinned independent-chunks
routine for the degenerate case, a differently written dense brute force, the identity with
sequential prefill that the prefix cache rests on, perturbation properties, and a hand-worked page
table."""
import os

import numpy as np

from oracle import attention as oa
from oracle import plan as op
from paper_2605_23296_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small(seed=3, workers=3, block_len=128, hq=4, hkv=2, d=64, steps=3, marker=16):
    return wl.prefix_aware(workers, block_len, hq, hkv, d, steps, seed=seed, marker_tokens=marker).materialise()


def brute_force_worker(q, k, v, k_pre, v_pre, scale):
    """One worker, written independently of the oracle: dense score matrix over [prefix; own]
    with an explicit mask (own token i sees the whole prefix and own tokens 0..i)."""
    n_pre, L, Hq = k_pre.shape[0], q.shape[0], q.shape[1]
    G = Hq // k.shape[1]
    qf = oa.bf16_bits_to_f64(q)
    kf = np.repeat(oa.bf16_bits_to_f64(np.concatenate([k_pre, k])), G, axis=1)
    vf = np.repeat(oa.bf16_bits_to_f64(np.concatenate([v_pre, v])), G, axis=1)
    s = np.einsum("ihc,jhc->hij", qf, kf) * scale
    cols = np.arange(n_pre + L)[None, :]
    hidden = cols > (n_pre + np.arange(L))[:, None]
    s = np.where(hidden[None], -np.inf, s)
    p = np.exp(s - s.max(axis=-1, keepdims=True))
    p /= p.sum(axis=-1, keepdims=True)
    return np.einsum("hij,jhc->ihc", p, vf)


def cu_of(w):
    return np.concatenate([[0], np.cumsum(w.own.block_lens)]).astype(np.int64)


def test_zero_prefix_is_independent_chunks():
    w = small()
    o, cu = w.own, cu_of(w)
    got = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, [0] * o.num_blocks, o.scale)
    np.testing.assert_array_equal(got, oa.prefill(o.q, o.k, o.v, cu, o.scale))


def test_matches_dense_brute_force():
    w = small(seed=5, workers=3, block_len=128, hq=4, hkv=2, d=64)
    o, cu = w.own, cu_of(w)
    got = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale)
    for b in range(o.num_blocks):
        n_pre = int(w.prefix_lens[b])
        want = brute_force_worker(o.q[cu[b]:cu[b + 1]], o.k[cu[b]:cu[b + 1]], o.v[cu[b]:cu[b + 1]],
                                  w.k_hist[:n_pre], w.v_hist[:n_pre], o.scale)
        np.testing.assert_allclose(got[cu[b]:cu[b + 1]], want, rtol=1e-11, atol=1e-13)


def test_without_markers_workers_reproduce_sequential_prefill():
    # What the prefix cache rests on: if worker b's own tokens are exactly history block b, its rows
    # are the rows of ONE causal pass over the whole history (sequential compaction's prefill).
    rng = np.random.default_rng(9)
    W, L, Hq, Hkv, d = 3, 48, 2, 1, 32
    bits = lambda shape: wl.f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))
    q, k, v = bits((W * L, Hq, d)), bits((W * L, Hkv, d)), bits((W * L, Hkv, d))
    cu = [b * L for b in range(W + 1)]
    got = oa.prefill_prefix_aware(q, k, v, cu, k, v, [b * L for b in range(W)], 0.3)
    np.testing.assert_array_equal(got, oa.prefill(q, k, v, [0, W * L], 0.3))


def test_only_the_visible_prefix_matters():
    w = small(seed=7)
    o, cu = w.own, cu_of(w)
    base = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale)
    b = 1                                    # worker 1 sees history tokens [0, prefix_lens[1])
    n_pre = int(w.prefix_lens[b])
    kh, vh = w.k_hist.copy(), w.v_hist.copy()
    kh[n_pre:] ^= 0x0100                      # history beyond its prefix: no effect on worker 1
    vh[n_pre:] ^= 0x0100
    out = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, kh, vh, w.prefix_lens, o.scale)
    np.testing.assert_array_equal(out[cu[b]:cu[b + 1]], base[cu[b]:cu[b + 1]])
    assert not np.array_equal(out[cu[2]:cu[3]], base[cu[2]:cu[3]])       # worker 2 sees those tokens
    vh = w.v_hist.copy()
    vh[n_pre - 1] ^= 0x0100                   # the last visible prefix token: every row of worker 1 moves
    out = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, vh, w.prefix_lens, o.scale)
    assert (np.abs(out[cu[b]:cu[b + 1]] - base[cu[b]:cu[b + 1]]).max(axis=(1, 2)) > 0).all()
    np.testing.assert_array_equal(out[cu[0]:cu[1]], base[cu[0]:cu[1]])   # worker 0 has no prefix


def test_constant_prefix_values_pull_rows_towards_them():
    # closed form: all keys zero -> uniform weights -> row i = mean of the prefix values and own values 0..i
    W, L, n_pre = 2, 5, 16
    k = np.zeros((W * L, 1, 8), dtype=np.uint16)
    q = wl.f32_to_bf16_bits(np.ones((W * L, 1, 8), dtype=np.float32))
    v = wl.f32_to_bf16_bits(np.arange(W * L, dtype=np.float32)[:, None, None] * np.ones((1, 1, 8), dtype=np.float32))
    kh = np.zeros((n_pre, 1, 8), dtype=np.uint16)
    vh = wl.f32_to_bf16_bits(np.full((n_pre, 1, 8), 100.0, dtype=np.float32))
    out = oa.prefill_prefix_aware(q, k, v, [0, L, 2 * L], kh, vh, [0, n_pre], 1.0)
    for i in range(L):
        np.testing.assert_allclose(out[i, 0], np.mean(np.arange(i + 1)), rtol=1e-14)
        own = np.arange(L, L + i + 1)
        np.testing.assert_allclose(out[L + i, 0], (100.0 * n_pre + own.sum()) / (n_pre + i + 1), rtol=1e-14)


def test_rows_selection_agrees_with_full_result():
    w = small(seed=8)
    o, cu = w.own, cu_of(w)
    full = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale)
    rows = [0, 5, int(cu[1]), int(cu[2]) - 1, int(cu[3]) - 1, int(cu[1]) + 7]
    part = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale, rows=rows)
    np.testing.assert_array_equal(part, full[rows])


def test_decode_step_is_last_row_of_the_extended_prompt():
    w = small(seed=4, steps=3)
    o, cu = w.own, cu_of(w)
    st = oa.PrefixDecodeState(o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.decode_steps)
    for t in range(o.decode_steps):
        st.append(o.k_dec[t], o.v_dec[t])
        got = st.decode(o.q_dec[t], o.scale)
        for b in range(o.num_blocks):
            own_k = np.concatenate([o.k[cu[b]:cu[b + 1]], o.k_dec[: t + 1, b]])
            own_v = np.concatenate([o.v[cu[b]:cu[b + 1]], o.v_dec[: t + 1, b]])
            own_q = np.concatenate([np.zeros((own_k.shape[0] - 1,) + o.q.shape[1:], dtype=np.uint16), o.q_dec[t, b][None]])
            n = own_k.shape[0]
            want = oa.prefill_prefix_aware(own_q, own_k, own_v, [0, n], w.k_hist, w.v_hist, [int(w.prefix_lens[b])],
                                           o.scale, rows=[n - 1])[0]
            np.testing.assert_allclose(got[b], want, rtol=1e-12, atol=1e-14)


def _read_golden(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            rows[key] = [int(x) for x in vals]
    return rows


def test_prefix_plan_matches_hand_worked_fixture():
    g = _read_golden("plan_prefix_small.txt")
    plan = op.build_plan([3, 2, 3], 1, 4, [8, 1, 5, 0, 9], 1, 2, 2, prefix_lens=[0, 4, 8], shared_pages=[6, 3])
    for key in ("cu_seqlens", "page_indptr", "page_indices", "seq_lens", "slot_mapping", "split_indptr"):
        assert plan[key] == g[key], key
    assert sum(plan["prefill_items"], []) == g["prefill_items"]
    assert sum(plan["decode_items"], []) == g["decode_items"]
    two = op.build_plan([3, 2, 3], 1, 4, [8, 1, 5, 0, 9], 1, 2, 2, prefix_lens=[0, 4, 8], shared_pages=[6, 3],
                        shared_chunk_pages=1)
    assert two["split_indptr"] == g["two_level_split_indptr"]
    assert sum(two["decode_items"], []) == g["two_level_decode_items"]
    for key in ("page_indptr", "page_indices", "seq_lens", "slot_mapping", "prefill_items"):
        assert two[key] == plan[key], key


def test_prefix_plan_invariants():
    w = small(seed=12, workers=4, block_len=256, steps=9)
    o = w.own
    P = o.page_size
    plan = op.build_plan(o.block_lens.tolist(), o.decode_steps, P, o.free_pages.tolist(), o.num_kv_heads, 256, 4,
                         prefix_lens=w.prefix_lens.tolist(), shared_pages=w.shared_pages.tolist())
    own_seen = []
    for b in range(o.num_blocks):
        pages = plan["page_indices"][plan["page_indptr"][b]:plan["page_indptr"][b + 1]]
        n_pre = int(w.prefix_lens[b]) // P
        assert pages[:n_pre] == w.shared_pages[:n_pre].tolist()          # every worker reads the same cached pages
        own_seen += pages[n_pre:]
        assert len(pages) - n_pre == -(-(int(o.block_lens[b]) + o.decode_steps) // P)
    assert own_seen == o.free_pages[: len(own_seen)].tolist()            # own pages: in order, each once
    assert not set(own_seen) & set(w.shared_pages.tolist())
    # own tokens never land in a shared page
    assert not {s // P for s in plan["slot_mapping"]} & set(w.shared_pages.tolist())
    assert plan["seq_lens"] == w.prefix_lens.tolist()


# ----------------------------------------------------------------------------
# the pins above can fail: plausible mistakes planted in copies of the oracle function (CPU only)
# ----------------------------------------------------------------------------

def _mutant(kind):
    """A copy of oracle.attention.prefill_prefix_aware's steps with one planted mistake."""
    def fn(q, k, v, cu_seqlens, k_hist, v_hist, prefix_lens, scale, rows=None):
        cu = [int(x) for x in cu_seqlens]
        out = np.empty(q.shape, dtype=np.float64)
        for w in range(len(cu) - 1):
            n_pre, lo, hi = int(prefix_lens[w]), cu[w], cu[w + 1]
            kh, vh = k_hist[:n_pre], v_hist[:n_pre]
            if kind == "prefix_from_the_end":          # the last n_pre history tokens instead of the first
                kh, vh = k_hist[k_hist.shape[0] - n_pre:], v_hist[v_hist.shape[0] - n_pre:]
            if kind == "prefix_one_short" and n_pre:   # drops the last visible history token
                kh, vh = kh[:-1], vh[:-1]
            if kind == "prefix_of_previous_worker":    # worker w reads worker w-1's prefix
                n_prev = int(prefix_lens[w - 1]) if w else 0
                kh, vh = k_hist[:n_prev], v_hist[:n_prev]
            if kind == "values_not_prefixed":          # keys see the prefix, values are shifted
                vh = np.roll(vh, 1, axis=0)
            m = kh.shape[0]
            pk, pv = np.concatenate([kh, k[lo:hi]]), np.concatenate([vh, v[lo:hi]])
            pq = np.concatenate([np.zeros((m,) + q.shape[1:], dtype=np.uint16), q[lo:hi]])
            first = m - 1 if kind == "rows_not_offset" and m else m    # the own rows start one row early
            out[lo:hi] = oa.prefill(pq, pk, pv, [0, m + hi - lo], scale, rows=list(range(first, first + hi - lo)))
        return out
    return fn


def _prefix_pins_hold(fn) -> bool:
    w = small(seed=5, workers=3, block_len=128, hq=4, hkv=2, d=64)
    o, cu = w.own, cu_of(w)
    got = fn(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale)
    for b in range(o.num_blocks):
        n_pre = int(w.prefix_lens[b])
        want = brute_force_worker(o.q[cu[b]:cu[b + 1]], o.k[cu[b]:cu[b + 1]], o.v[cu[b]:cu[b + 1]],
                                  w.k_hist[:n_pre], w.v_hist[:n_pre], o.scale)
        if not np.allclose(got[cu[b]:cu[b + 1]], want, rtol=1e-11, atol=1e-13):
            return False
    return True


def test_prefix_pins_reject_planted_mistakes():
    assert _prefix_pins_hold(oa.prefill_prefix_aware)
    for kind in ("prefix_from_the_end", "prefix_one_short", "prefix_of_previous_worker", "values_not_prefixed",
                 "rows_not_offset"):
        assert not _prefix_pins_hold(_mutant(kind)), kind
    assert _prefix_pins_hold(_mutant("none"))     # the copy without a mistake passes, so the copies are faithful
