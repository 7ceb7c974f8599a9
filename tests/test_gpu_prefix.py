"""Parity of the prefix-aware layout (paper, Section 4: a worker's prompt is the cached history up to
its block, then its own tokens) on the CUDA path, through the C-ABI, against the CPU oracle: page
table and pool bytes bit-exact, attention within max-abs 1e-2 / mean-abs 1e-3."""
import numpy as np
import pytest

from _util import assert_attention_close, pool_rows
from oracle import attention as oa
from oracle import plan as op
from paper_2605_23296_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _dev(bits):
    from paper_2605_23296_b200.session import bits_to_tensor
    return bits_to_tensor(bits, "cuda:0")


def _bits(t):
    from paper_2605_23296_b200.session import tensor_to_bits
    return tensor_to_bits(t)


def _sessions(w, poison=True, pages_per_split=0, q_tile_rows=0):
    """(history session or None, workers' session): the history is cached first, through a plan of
    its own that owns the shared pages; the workers' plan then reads those pages."""
    import torch
    from paper_2605_23296_b200.session import CompactionSession
    o = w.own
    shape = (w.num_pages, o.num_kv_heads, o.page_size, o.head_dim)
    fill = float("nan") if poison else 0.0
    pools = (torch.full(shape, fill, dtype=torch.bfloat16, device="cuda:0"),
             torch.full(shape, fill, dtype=torch.bfloat16, device="cuda:0"))
    hist = None
    if w.hist_tokens:
        hist = CompactionSession([w.hist_tokens], 0, o.num_q_heads, o.num_kv_heads, o.head_dim, w.shared_pages,
                                 w.num_pages, scale=o.scale, pools=pools)
        hist.append_prefill(_dev(w.k_hist), _dev(w.v_hist))
    s = CompactionSession(o.block_lens, o.decode_steps, o.num_q_heads, o.num_kv_heads, o.head_dim, o.free_pages,
                          w.num_pages, scale=o.scale, pages_per_split=pages_per_split, q_tile_rows=q_tile_rows,
                          prefix_lens=w.prefix_lens, shared_pages=w.shared_pages, pools=pools)
    return hist, s


def _cu(o):
    return np.concatenate([[0], np.cumsum(o.block_lens.astype(np.int64))])


def run_event(w, pages_per_split=0, q_tile_rows=0, fused_every=2):
    from paper_2605_23296_b200 import binding as B
    o = w.own
    cu = _cu(o)
    hist, s = _sessions(w, pages_per_split=pages_per_split, q_tile_rows=q_tile_rows)
    try:
        # page table: bit-exact with the restated rules
        C = s.export(B.ARR_SPLIT_PAGES).tolist()
        CH = s.param(B.PARAM_SHARED_CHUNK_PAGES)
        ref = op.build_plan(o.block_lens.tolist(), o.decode_steps, o.page_size, o.free_pages.tolist(), o.num_kv_heads,
                            s.param(B.PARAM_Q_TILE_ROWS), C, prefix_lens=w.prefix_lens.tolist(),
                            shared_pages=w.shared_pages.tolist(), shared_chunk_pages=CH)
        even = s.param(B.PARAM_DECODE_EVEN_CUT)
        for which, key in [(B.ARR_PAGE_INDPTR, "page_indptr"), (B.ARR_PAGE_INDICES, "page_indices"),
                           (B.ARR_SLOT_MAPPING, "slot_mapping"), (B.ARR_SEQ_LENS, "seq_lens"),
                           (B.ARR_SPLIT_INDPTR, "split_indptr"), (B.ARR_DECODE_ITEMS, "decode_items")]:
            if even and key in ("split_indptr", "decode_items"):
                continue    # the even cut of the decode pages is the planner's free choice (host tests check it)
            got = s.export(which)
            assert np.array_equal(got, np.asarray(ref[key], dtype=np.int32).reshape(got.shape)), key
        # prefill of the own tokens over prefix + own tokens
        k, v = _dev(o.k), _dev(o.v)
        out = s.prefill(_dev(o.q), k, v)
        want = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale)
        assert s.status() == 0
        assert_attention_close(_bits(out), want, f"{o.name} prefix-aware prefill")
        # the own tokens go behind the prefix, the shared pages keep the history bit for bit
        s.append_prefill(k, v)
        kp, vp = pool_rows(_bits(s.k_pool)), pool_rows(_bits(s.v_pool))
        P = o.page_size
        for i, slot in enumerate(ref["slot_mapping"]):
            assert np.array_equal(kp[slot // P, :, slot % P], o.k[i]) and np.array_equal(vp[slot // P, :, slot % P], o.v[i])
        for t in range(w.hist_tokens):
            page = int(w.shared_pages[t // P])
            assert np.array_equal(kp[page, :, t % P], w.k_hist[t]) and np.array_equal(vp[page, :, t % P], w.v_hist[t])
        # decode over shared prefix pages + own pages
        st = oa.PrefixDecodeState(o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.decode_steps)
        for t in range(o.decode_steps):
            st.append(o.k_dec[t], o.v_dec[t])
            if fused_every and t % fused_every == 0:
                got = s.decode_append(_dev(o.q_dec[t]), _dev(o.k_dec[t]), _dev(o.v_dec[t]))
            else:
                s.append(_dev(o.k_dec[t]), _dev(o.v_dec[t]))
                got = s.decode(_dev(o.q_dec[t]))
            assert_attention_close(_bits(got), st.decode(o.q_dec[t], o.scale), f"{o.name} prefix-aware decode step {t}")
        assert s.status() == 0
        assert np.array_equal(s.export(B.ARR_SEQ_LENS), w.prefix_lens + o.block_lens + o.decode_steps)
    finally:
        s.close()
        if hist is not None:
            hist.close()


@pytest.mark.parametrize("workers,block_len,hq,hkv,d", [(3, 128, 4, 1, 64), (4, 256, 8, 2, 128), (3, 384, 8, 8, 128),
                                                        (5, 128, 16, 2, 64), (4, 128, 6, 2, 128)])
def test_prefix_aware_event(workers, block_len, hq, hkv, d):
    run_event(wl.prefix_aware(workers, block_len, hq, hkv, d, steps=5, seed=workers + d).materialise())


def test_prefix_aware_markers_make_ragged_own_lengths():
    # own lengths that are not multiples of anything: partial last q tile, partial last page
    run_event(wl.prefix_aware(3, 256, 8, 2, 128, steps=3, seed=31, marker_tokens=37).materialise())


@pytest.mark.parametrize("q_tile_rows", [128, 256])
def test_prefix_aware_both_work_item_sizes(q_tile_rows):
    run_event(wl.prefix_aware(3, 256, 4, 2, 64, steps=2, seed=17).materialise(), q_tile_rows=q_tile_rows)


def test_prefix_aware_small_decode_splits():
    run_event(wl.prefix_aware(3, 256, 8, 2, 128, steps=4, seed=23).materialise(), pages_per_split=3)


def test_decode_with_two_worker_groups():
    # G = 8: sixteen workers fill the 128 rows of a shared-scan item, twenty workers need two groups
    run_event(wl.prefix_aware(20, 128, 16, 2, 128, steps=3, seed=29).materialise())


def test_prefix_ends_inside_a_shared_chunk():
    # 136-page blocks against 16-page chunks (more pages than the scan's ring has stages): the prefixes of
    # workers 1 and 3 end in the middle of a chunk, so the rows of one shared-scan item see different
    # numbers of its keys, and the ring of stages is refilled while the warps are at different pages
    w = wl.prefix_aware(5, 2176, 8, 8, 64, steps=2, seed=37).materialise()
    from paper_2605_23296_b200 import binding as B
    hist, s = _sessions(w)
    try:
        ch = s.param(B.PARAM_SHARED_CHUNK_PAGES)
        assert ch >= 16 and any((int(x) // 16) % ch for x in w.prefix_lens)
    finally:
        s.close()
        hist.close()
    run_event(w)


def test_decode_long_shared_chunks_sampled_steps():
    # 8 workers x 4096-token blocks, d = 128: chunks of 40 pages against a ring of 8 stages
    w = wl.prefix_aware(8, 4096, 32, 8, 128, steps=3, seed=43).materialise()
    o = w.own
    cu = _cu(o)
    hist, s = _sessions(w, poison=False)
    try:
        from paper_2605_23296_b200 import binding as B
        assert s.param(B.PARAM_SHARED_CHUNK_PAGES) > 8
        s.append_prefill(_dev(o.k), _dev(o.v))
        st = oa.PrefixDecodeState(o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.decode_steps)
        for t in range(o.decode_steps):
            st.append(o.k_dec[t], o.v_dec[t])
            got = s.decode_append(_dev(o.q_dec[t]), _dev(o.k_dec[t]), _dev(o.v_dec[t]))
            assert_attention_close(_bits(got), st.decode(o.q_dec[t], o.scale), f"long shared chunks, step {t}")
        assert s.status() == 0
    finally:
        s.close()
        hist.close()


def test_single_worker_has_no_prefix_and_equals_plain_prefill():
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.prefix_aware(1, 256, 8, 2, 128, steps=0, seed=5).materialise()
    o = w.own
    _, s = _sessions(w)
    plain = CompactionSession(o.block_lens, 0, o.num_q_heads, o.num_kv_heads, o.head_dim, o.free_pages, w.num_pages,
                              scale=o.scale)
    try:
        a = s.prefill(_dev(o.q), _dev(o.k), _dev(o.v))
        b = plain.prefill(_dev(o.q), _dev(o.k), _dev(o.v))
        assert np.array_equal(_bits(a), _bits(b))
    finally:
        s.close()
        plain.close()


def test_long_prefix_sampled_rows():
    # 8 workers x 2048-token blocks: prefixes up to 14336 tokens (112 tiles); rows sampled per worker
    w = wl.prefix_aware(8, 2048, 32, 8, 128, steps=0, seed=41).materialise(with_decode=False)
    o = w.own
    cu = _cu(o)
    hist, s = _sessions(w, poison=False)
    try:
        out = _bits(s.prefill(_dev(o.q), _dev(o.k), _dev(o.v)))
        assert s.status() == 0
        rng = np.random.default_rng(0)
        rows = []
        for b in range(o.num_blocks):
            L = int(o.block_lens[b])
            rows += [int(cu[b]) + r for r in sorted({0, 1, 127, 128, 129, 255, 256, L - 1} | set(rng.integers(0, L, 6).tolist()))]
        want = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale, rows=rows)
        assert_attention_close(out[rows], want, "long prefix, sampled rows")
    finally:
        s.close()
        hist.close()


def test_entry_points_and_layouts_do_not_mix():
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.prefix_aware(2, 128, 4, 2, 64, steps=1, seed=3).materialise()
    o = w.own
    hist, s = _sessions(w)
    plain = CompactionSession(o.block_lens, 1, o.num_q_heads, o.num_kv_heads, o.head_dim, o.free_pages, w.num_pages,
                              scale=o.scale, pools=(s.k_pool, s.v_pool))
    try:
        q, k, v = _dev(o.q), _dev(o.k), _dev(o.v)
        out = _dev(np.zeros_like(o.q))
        # a plan with cached prefixes needs the pools: the plain prefill calls refuse it
        assert B.cpa_prefill(s.plan, q, k, v, out, None, 0) == B.CPA_EINVAL
        assert B.cpa_prefill_variant(s.plan, q, k, v, out, 0, 1) == B.CPA_EINVAL
        assert B.cpa_prefill_prefix(s.plan, q, k, v, None, s.v_pool, out, 0) == B.CPA_EINVAL
        # a plan without prefixes through the prefix entry point reads nothing from the pools
        a = plain.prefill(q, k, v)
        b = _dev(np.zeros_like(o.q))
        assert B.cpa_prefill_prefix(plain.plan, q, k, v, plain.k_pool, plain.v_pool, b, plain._stream()) == B.CPA_OK
        assert plain.status() == 0
        assert np.array_equal(_bits(a), _bits(b))
        assert plain.param(B.PARAM_SHARED_CHUNK_PAGES) == 0 and s.param(B.PARAM_SHARED_CHUNK_PAGES) >= 8
    finally:
        s.close()
        plain.close()
        hist.close()


def test_prefill_only_event_and_single_token_workers():
    # T = 0 (no decode), and workers whose own part is a single token behind a long prefix
    w = wl.prefix_aware(3, 256, 8, 2, 128, steps=0, seed=13, own_len=1).materialise(with_decode=False)
    o = w.own
    cu = _cu(o)
    hist, s = _sessions(w)
    try:
        out = s.prefill(_dev(o.q), _dev(o.k), _dev(o.v))
        want = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale)
        assert s.status() == 0
        assert_attention_close(_bits(out), want, "single own token behind a prefix")
    finally:
        s.close()
        hist.close()


def test_decode_entry_points_agree_on_a_prefix_plan():
    # separate append + cpa_decode, the fused step and the static-scratch variant over shared prefix pages
    import torch
    from paper_2605_23296_b200 import binding as B
    w = wl.prefix_aware(4, 256, 8, 2, 128, steps=2, seed=19).materialise()
    o = w.own
    hist, s = _sessions(w)
    try:
        s.append_prefill(_dev(o.k), _dev(o.v))
        s.append(_dev(o.k_dec[0]), _dev(o.v_dec[0]))
        q = _dev(o.q_dec[0])
        want = s.decode(q)
        again = s.decode(q)
        assert np.array_equal(_bits(want), _bits(again))          # the merge tickets reset themselves
        got = torch.full_like(want, 7.0)
        assert B.cpa_decode_static(s.plan, q, s.k_pool, s.v_pool, got, s._stream()) == B.CPA_OK
        assert s.status() == 0
        assert np.array_equal(_bits(got), _bits(want))
    finally:
        s.close()
        hist.close()


def test_full_prefix8b_sampled():
    # the configuration `bench.py --config prefix8b` times, in its launch configuration: 16 workers x
    # (8192 + 16) own tokens over a cached history of 15 x 8192 tokens; prefill rows and decode outputs
    # are checked on samples the oracle computes one by one
    w = wl.prefix_aware(16, 8192, 32, 8, 128, 2, seed=11, permute_pages=False).materialise()
    o = w.own
    cu = _cu(o)
    hist, s = _sessions(w, poison=False)
    try:
        k, v = _dev(o.k), _dev(o.v)
        out = _bits(s.prefill(_dev(o.q), k, v))
        assert s.status() == 0
        rng = np.random.default_rng(1)
        rows = []
        for b in (0, 1, 7, 15):
            L = int(o.block_lens[b])
            rows += [int(cu[b]) + r for r in sorted({0, 127, 128, 255, 256, L - 1} | set(rng.integers(0, L, 2).tolist()))]
        want = oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale, rows=rows)
        assert_attention_close(out[rows], want, "prefix8b prefill, sampled rows")
        s.append_prefill(k, v)
        st = oa.PrefixDecodeState(o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.decode_steps)
        for t in range(o.decode_steps):
            st.append(o.k_dec[t], o.v_dec[t])
            got = _bits(s.decode_append(_dev(o.q_dec[t]), _dev(o.k_dec[t]), _dev(o.v_dec[t])))
            blocks = [0, 1, 8, 15]
            want = st.decode(o.q_dec[t], o.scale, blocks=blocks)
            assert_attention_close(got[blocks], want[blocks], f"prefix8b decode step {t}, sampled workers")
        assert s.status() == 0
    finally:
        s.close()
        hist.close()
