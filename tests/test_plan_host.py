"""Host-side checks that need no GPU: the planner against the independent Python
restatement (bit-exact), error codes, and the exported C symbols."""
import os
import re

import numpy as np
import pytest

from oracle import plan as op
from paper_2605_23296_b200 import binding as B
from paper_2605_23296_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def make_plan(w, pages_per_split=0, free=None, num_sms=0):
    cfg = B.cpa_config(w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size, w.scale, 0,
                       pages_per_split, num_sms)
    if free is None:
        free = np.arange(w.num_pages, dtype=np.int32)
    return B.cpa_plan_create(cfg, w.block_lens, w.decode_steps, free), free


def check_schedule(sched, ctas, prefill_items, block_lens, q_rows, num_q_heads, num_kv_heads, prefix_lens=None,
                   balance=None):
    """The deal of prefill units (item, query head) to persistent CTAs has many valid answers, so it
    is checked by what is fixed: every unit exactly once; the units of round r are units
    [r * ctas, (r + 1) * ctas) of the kv-head-major list (kv head, then item, then head inside the
    group), which is what keeps concurrently running CTAs on the same few K/V ranges; and, where
    `balance` is given, the most loaded CTA streams at most `balance` times the mean number of KV
    tiles (128 keys each; counted here from the definition of a unit, not from the planner's cost)."""
    table = np.asarray(sched).reshape(-1, ctas)
    n_items, G = len(prefill_items), num_q_heads // num_kv_heads
    n_units = n_items * num_q_heads
    codes = table[table >= 0]
    assert sorted(codes.tolist()) == list(range(n_units))
    item, head = table // num_q_heads, table % num_q_heads
    pos = (head // G) * (n_items * G) + item * G + head % G          # place in the kv-head-major list
    for r in range(table.shape[0]):
        valid = table[r] >= 0
        lo = r * ctas
        assert sorted(pos[r][valid].tolist()) == list(range(lo, min(lo + ctas, n_units))), f"round {r}"
    if balance is not None:
        tiles = np.zeros(n_items, dtype=np.int64)
        for i, (b, t) in enumerate(prefill_items):
            last_row = min((t + 1) * q_rows, int(block_lens[b]))       # keys its last row sees inside the block
            pre = int(prefix_lens[b]) if prefix_lens is not None else 0
            tiles[i] = pre // 128 + -(-last_row // 128)
        load = np.where(table >= 0, tiles[np.clip(item, 0, n_items - 1)], 0).sum(axis=0)
        assert load.max() <= balance * load.mean(), (load.max(), load.mean())


def check_decode_cut(plan, own_pages, num_kv_heads, n_fixed=None):
    """The decode splits, whichever way the planner cut them: the splits of a block tile its own pages in order
    without gaps, all but the first and the last have the block's split size, every (block, kv head, split) is an
    item exactly once, and the launch is one wave at most."""
    B_ = len(own_pages)
    n_fixed = n_fixed or [0] * B_
    indptr = B.cpa_plan_export(plan, B.ARR_SPLIT_INDPTR)
    ranges = B.cpa_plan_export(plan, B.ARR_SPLIT_RANGES)
    C = B.cpa_plan_export(plan, B.ARR_SPLIT_PAGES)
    want_items = set()
    for b in range(B_):
        rows = ranges[indptr[b] + n_fixed[b]:indptr[b + 1]]
        assert len(rows) >= 1 and rows[0][0] == 0
        pos = 0
        for s, (first, pages) in enumerate(rows.tolist()):
            assert first == pos and pages >= 1
            if 0 < s < len(rows) - 1:
                assert pages == C[b]
            if s == len(rows) - 1 and s > 0:
                assert pages <= C[b]
            pos += pages
            want_items |= {(b, g, s) for g in range(num_kv_heads)}
        assert pos == own_pages[b]
    items = [tuple(x) for x in B.cpa_plan_export(plan, B.ARR_DECODE_ITEMS).tolist()]
    assert len(items) == len(set(items)) and set(items) == want_items
    sms = B.cpa_plan_param(plan, B.PARAM_NUM_SMS)
    assert 1 <= B.cpa_plan_param(plan, B.PARAM_DECODE_CTAS) <= 3 * sms


def check_against_oracle(w, pages_per_split=0, permute=False, balance=None):
    free = None
    if permute:
        free = np.random.default_rng(w.seed).permutation(w.num_pages).astype(np.int32)
    plan, free = make_plan(w, pages_per_split, free)
    try:
        C = B.cpa_plan_export(plan, B.ARR_SPLIT_PAGES).tolist()      # pages per split, per block
        assert max(C) == B.cpa_plan_param(plan, B.PARAM_PAGES_PER_SPLIT)
        if pages_per_split:
            assert C == [pages_per_split] * w.num_blocks
        M = B.cpa_plan_param(plan, B.PARAM_Q_TILE_ROWS)
        ref = op.build_plan(w.block_lens.tolist(), w.decode_steps, w.page_size, free.tolist(),
                            w.num_kv_heads, M, C)
        pairs = [(B.ARR_CU_SEQLENS, "cu_seqlens"), (B.ARR_PAGE_INDPTR, "page_indptr"),
                 (B.ARR_PAGE_INDICES, "page_indices"), (B.ARR_SEQ_LENS, "seq_lens"),
                 (B.ARR_SLOT_MAPPING, "slot_mapping"), (B.ARR_PREFILL_ITEMS, "prefill_items"),
                 (B.ARR_DECODE_ITEMS, "decode_items"), (B.ARR_SPLIT_INDPTR, "split_indptr")]
        even = B.cpa_plan_param(plan, B.PARAM_DECODE_EVEN_CUT)
        assert not (even and pages_per_split)               # a given split size is kept
        for which, key in pairs:
            if even and key in ("decode_items", "split_indptr"):
                continue    # the even cut is a free choice of the planner: checked by what is fixed (below)
            got = B.cpa_plan_export(plan, which)
            want = np.asarray(ref[key], dtype=np.int32).reshape(got.shape)
            assert np.array_equal(got, want), key
        own_pages = (-(-(w.block_lens.astype(np.int64) + w.decode_steps) // w.page_size)).tolist()
        check_decode_cut(plan, own_pages, w.num_kv_heads)
        # the deal of prefill units to persistent CTAs: a free choice, checked by its invariants
        ctas = B.cpa_plan_param(plan, B.PARAM_PREFILL_CTAS)
        n_units = len(ref["prefill_items"]) * w.num_q_heads
        assert ctas == min(148 // 2 if M == 512 else 148, n_units)      # 512-row items run on pairs of CTAs
        check_schedule(B.cpa_plan_export(plan, B.ARR_PREFILL_SCHED), ctas, ref["prefill_items"], w.block_lens, M,
                       w.num_q_heads, w.num_kv_heads, balance=balance)
        assert B.cpa_plan_param(plan, B.PARAM_NUM_BLOCKS) == w.num_blocks
        assert B.cpa_plan_param(plan, B.PARAM_TOTAL_TOKENS) == w.total_tokens
        assert B.cpa_plan_param(plan, B.PARAM_PAGES_USED) == w.pages_needed
        assert even or B.cpa_plan_param(plan, B.PARAM_TOTAL_SPLITS) == ref["split_indptr"][-1]
        assert B.cpa_plan_param(plan, B.PARAM_MAX_NEW_TOKENS) == w.decode_steps
        rows = B.cpa_plan_param(plan, B.PARAM_TOTAL_SPLITS) * w.num_q_heads
        assert B.cpa_plan_param(plan, B.PARAM_DECODE_WORKSPACE_BYTES) >= rows * (w.head_dim + 2) * 4
        return C, even
    finally:
        B.cpa_plan_destroy(plan)


@pytest.mark.parametrize("pps", [0, 1, 3, 8])
def test_plan_bit_exact_tiny(pps):
    check_against_oracle(wl.tiny(), pps, permute=True)


def test_plan_bit_exact_edge_lengths():
    w = wl.custom([1, 15, 16, 17, 127, 128, 129, 1000], 8, 2, 64, steps=5)
    check_against_oracle(w, 0, permute=True)
    w = wl.custom([4097], 4, 4, 128, steps=0)
    check_against_oracle(w, 2)


@pytest.mark.parametrize("name", ["dense8b", "ragged", "moe120b"])
def test_plan_bit_exact_full_configs(name):
    w = wl.CONFIGS[name]()
    C, even = check_against_oracle(w, 0, permute=(name == "ragged"), balance=1.05)
    if even:
        return      # the even cut has its own invariants (check_decode_cut)
    pages = (w.block_lens.astype(np.int64) + w.decode_steps + 15) // 16
    n_items = int((w.num_kv_heads * -(-pages // np.asarray(C))).sum())
    assert n_items <= 3 * 148                       # one wave of three CTAs per SM
    assert n_items + w.num_kv_heads > 3 * 148 or max(C) <= 4
    sizes = -(-pages // -(-pages // np.asarray(C)))
    # greedy rule: the largest split could not be halved any more within the wave, and every
    # split that was made is at least as large as half the largest remaining one
    n_splits = -(-pages // np.asarray(C))
    assert (sizes[n_splits > 1] * 2 >= sizes.max() - 1).all()


@pytest.mark.parametrize("nb", [1, 2, 8, 64])
def test_plan_bit_exact_split_sweep(nb):
    check_against_oracle(wl.split_sweep(nb), 0)


def test_even_cut_for_equal_blocks_that_do_not_divide_the_wave():
    # 64 x 2048 tokens, 8 kv heads: 512 (block, head) pairs against 444 CTAs of a wave.  One split per block leaves 68
    # CTAs with two items; the even cut gives every CTA the same pages.
    w = wl.split_sweep(64)
    plan, _ = make_plan(w, 0)
    try:
        assert B.cpa_plan_param(plan, B.PARAM_DECODE_EVEN_CUT) == 1
        pages = (-(-(w.block_lens.astype(np.int64) + w.decode_steps) // 16)).tolist()
        check_decode_cut(plan, pages, w.num_kv_heads)
        ctas = B.cpa_plan_param(plan, B.PARAM_DECODE_CTAS)
        C = B.cpa_plan_param(plan, B.PARAM_PAGES_PER_SPLIT)
        assert ctas % w.num_kv_heads == 0 and ctas <= 444
        assert C == -(-sum(pages) // (ctas // w.num_kv_heads))          # equal ranges over all pages laid end to end
        ranges = B.cpa_plan_export(plan, B.ARR_SPLIT_RANGES)
        assert ranges[:, 1].max() <= C + C // 16 + 2
    finally:
        B.cpa_plan_destroy(plan)
    # a split size given by the caller is kept as it is
    plan, _ = make_plan(w, 100)
    assert B.cpa_plan_param(plan, B.PARAM_DECODE_EVEN_CUT) == 0
    B.cpa_plan_destroy(plan)


def test_auto_split_aims_at_the_sm_count():
    w = wl.dense8b()
    plan_a, _ = make_plan(w, 0, num_sms=148)
    plan_b, _ = make_plan(w, 0, num_sms=16)
    try:
        ca = B.cpa_plan_param(plan_a, B.PARAM_PAGES_PER_SPLIT)
        cb = B.cpa_plan_param(plan_b, B.PARAM_PAGES_PER_SPLIT)
        assert cb >= ca
        assert B.cpa_plan_export(plan_a, B.ARR_DECODE_ITEMS).shape[0] <= 3 * 148
        assert B.cpa_plan_export(plan_b, B.ARR_DECODE_ITEMS).shape[0] == 64      # one split per (block, head)
    finally:
        B.cpa_plan_destroy(plan_a)
        B.cpa_plan_destroy(plan_b)


def test_plan_errors():
    ok = B.cpa_config(8, 2, 64, 16, 0.125, 0, 0, 0)
    free = np.arange(100, dtype=np.int32)

    def rc(cfg=ok, lens=(40, 50), T=4, fr=free):
        status, handle = B.cpa_plan_create(cfg, lens, T, fr, check=False)
        assert status != 0 and not handle
        return status

    assert rc(lens=(40, 0)) == B.CPA_EINVAL                      # zero-length block
    assert rc(lens=(40, -3)) == B.CPA_EINVAL
    assert rc(T=-1) == B.CPA_EINVAL
    assert rc(fr=np.arange(5, dtype=np.int32)) == B.CPA_ENOSPC   # too few pages
    assert rc(fr=np.array([0, 1, 2, -4, 5, 6, 7, 8], dtype=np.int32)) == B.CPA_EINVAL
    # the largest page id: (2^31 - 1) / max(64, 32 * kv heads), so that a pool's rows keep 32-bit coordinates
    top = (2 ** 31 - 1) // 64
    assert rc(fr=np.array([0, 1, 2, top + 1, 5, 6, 7, 8], dtype=np.int32)) == B.CPA_EINVAL
    handle = B.cpa_plan_create(ok, (40, 50), 4, np.array([0, 1, 2, top, 5, 6, 7, 8], dtype=np.int32))
    B.cpa_plan_destroy(handle)
    wide = B.cpa_config(32, 8, 64, 16, 0.125, 0, 0, 0)
    top8 = (2 ** 31 - 1) // 256
    assert rc(cfg=wide, fr=np.array([0, 1, 2, top8 + 1, 5, 6, 7, 8], dtype=np.int32)) == B.CPA_EINVAL
    handle = B.cpa_plan_create(wide, (40, 50), 4, np.array([0, 1, 2, top8, 5, 6, 7, 8], dtype=np.int32))
    B.cpa_plan_destroy(handle)
    assert rc(cfg=B.cpa_config(8, 3, 64, 16, 0.125, 0, 0, 0)) == B.CPA_EINVAL        # 8 % 3
    assert rc(cfg=B.cpa_config(8, 2, 96, 16, 0.125, 0, 0, 0)) == B.CPA_EUNSUPPORTED  # head_dim
    assert rc(cfg=B.cpa_config(8, 2, 64, 32, 0.125, 0, 0, 0)) == B.CPA_EUNSUPPORTED  # page size
    assert rc(cfg=B.cpa_config(16, 1, 64, 16, 0.125, 0, 0, 0)) == B.CPA_EUNSUPPORTED # G = 16
    assert rc(cfg=B.cpa_config(8, 2, 64, 16, 0.0, 0, 0, 0)) == B.CPA_EINVAL          # scale
    assert rc(cfg=B.cpa_config(8, 2, 64, 16, 0.125, 0, 1025, 0)) == B.CPA_EUNSUPPORTED # split size
    with pytest.raises(B.CpaError):
        B.cpa_plan_create(ok, (40, 0), 4, free)
    # T = 0 is allowed (prefill only)
    plan = B.cpa_plan_create(ok, (40, 50), 0, free)
    B.cpa_plan_destroy(plan)


def test_compute_calls_before_upload_report_state_error():
    plan = B.cpa_plan_create(B.cpa_config(8, 2, 64, 16, 0.125, 0, 0, 0), (40, 50), 4,
                             np.arange(100, dtype=np.int32))
    try:
        fake = 4096  # a 16-byte aligned non-null address; never dereferenced before the state check
        assert B.cpa_prefill(plan, fake, fake, fake, fake + 16) == B.CPA_ESTATE
        assert B.cpa_kv_append(plan, fake, fake, None, fake, fake) == B.CPA_ESTATE
        assert B.cpa_decode(plan, fake, fake, fake, fake, fake) == B.CPA_ESTATE
        assert B.cpa_plan_status(plan) == B.CPA_ESTATE
        assert B.cpa_prefill(plan, None, fake, fake, fake) == B.CPA_EINVAL
        assert B.cpa_prefill(plan, fake + 2, fake, fake, fake + 16) == B.CPA_EINVAL   # misaligned
        assert B.cpa_decode(plan, fake, fake, fake, fake, None) == B.CPA_EINVAL
    finally:
        B.cpa_plan_destroy(plan)
    for code in range(0, -7, -1):
        assert B.cpa_strerror(code) and B.cpa_strerror(code) != "unknown status"
    assert B.cpa_strerror(-99) == "unknown status"


def test_library_exports_every_declared_symbol():
    import ctypes
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names |= set(re.findall(r"CPA_API\s+[\w\s\*]*?\b(cpa_\w+)\s*\(", text))
    assert {"cpa_plan_create", "cpa_prefill", "cpa_kv_append", "cpa_decode"} <= names
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in sorted(names):
        assert hasattr(lib, n), n


# ----------------------------------------------------------------------------
# chunked prefill: the steps of the schedule
# ----------------------------------------------------------------------------

@pytest.mark.parametrize("lens,C,T,r", [([300, 100, 50], 128, 2, 1), ([300, 100, 50], 128, 3, 2),
                                         ([16384, 2048, 2048, 2048, 2048], 2048, 256, 16),
                                         ([1, 129, 128, 1000], 128, 3, 1), ([700], 256, 0, 4)])
def test_chunked_plan_steps_bit_exact(lens, C, T, r):
    cfg = B.cpa_config(8, 2, 128, 16, 0.088, 0, 0, 0)
    pages = sum(-(-(L + T) // 16) for L in lens)
    plan = B.cpa_plan_create_chunked(cfg, lens, T, C, np.arange(pages, dtype=np.int32), decode_steps_per_chunk=r)
    try:
        ref = op.mixed_schedule(lens, C, T, r)
        assert B.cpa_plan_param(plan, B.PARAM_NUM_STEPS) == len(ref)
        assert B.cpa_plan_param(plan, B.PARAM_CHUNK_TOKENS) == C
        assert B.cpa_plan_param(plan, B.PARAM_DECODE_STEPS_PER_CHUNK) == r
        n_chunks = B.cpa_plan_param(plan, B.PARAM_CHUNK_STEPS)
        assert n_chunks == sum(1 for st in ref if st["prefill"])
        start = B.cpa_plan_export(plan, B.ARR_DEC_START).tolist()
        rows = B.cpa_plan_export(plan, B.ARR_CHUNK_ROWS).reshape(n_chunks, len(lens) + 1)
        for s, st in enumerate(ref):
            assert [b for b in range(len(lens)) if 0 <= s - start[b] < T] == st["decode"]
            if s % r == 0 and s // r < n_chunks:
                c = s // r
                per_block = np.diff(rows[c]).tolist()
                want = [0] * len(lens)
                for b, first, n in st["prefill"]:
                    assert first == c * C
                    want[b] = n
                assert per_block == want and rows[c][0] == 0
            else:
                assert not st["prefill"]
        # everything the whole-block calls use is the ordinary plan's
        cfg256 = B.cpa_config(8, 2, 128, 16, 0.088, B.cpa_plan_param(plan, B.PARAM_Q_TILE_ROWS), 0, 0)
        plain = B.cpa_plan_create(cfg256, lens, T, np.arange(pages, dtype=np.int32))
        for which in (B.ARR_CU_SEQLENS, B.ARR_PAGE_INDICES, B.ARR_SLOT_MAPPING, B.ARR_PREFILL_ITEMS, B.ARR_DECODE_ITEMS):
            assert np.array_equal(B.cpa_plan_export(plan, which), B.cpa_plan_export(plain, which))
        B.cpa_plan_destroy(plain)
        sms = B.cpa_plan_param(plan, B.PARAM_NUM_SMS)
        assert 1 <= B.cpa_plan_param(plan, B.PARAM_DECODE_SMS) < sms
    finally:
        B.cpa_plan_destroy(plan)


def test_prefix_chunked_plan_is_the_prefix_plan_with_the_chunk_schedule():
    # Section 4.2 runs prefix caching and chunked prefill together: pages, slots, lengths and the two-level
    # decode cut are the prefix plan's, the steps are those of the chunk schedule over the own lengths
    cfg = B.cpa_config(8, 2, 128, 16, 0.088, 0, 0, 0)
    own, pre, T, C, r = [272, 700, 129, 50], [0, 256, 512, 768], 3, 256, 2
    shared = np.arange(100, 100 + 48, dtype=np.int32)
    free = np.arange(sum(-(-(L + T) // 16) for L in own), dtype=np.int32)
    plan = B.cpa_plan_create_prefix_chunked(cfg, own, pre, shared, T, C, free, decode_steps_per_chunk=r)
    try:
        ref = op.mixed_schedule(own, C, T, r)
        assert B.cpa_plan_param(plan, B.PARAM_NUM_STEPS) == len(ref)
        n_chunks = B.cpa_plan_param(plan, B.PARAM_CHUNK_STEPS)
        rows = B.cpa_plan_export(plan, B.ARR_CHUNK_ROWS).reshape(n_chunks, len(own) + 1)
        for c in range(n_chunks):
            want = [0] * len(own)
            for b, first, n in ref[c * r]["prefill"]:
                want[b] = n
            assert np.diff(rows[c]).tolist() == want
        assert B.cpa_plan_export(plan, B.ARR_DEC_START).tolist() == [-(-L // C) * r for L in own]
        cfgq = B.cpa_config(8, 2, 128, 16, 0.088, B.cpa_plan_param(plan, B.PARAM_Q_TILE_ROWS), 0, 0)
        plain = B.cpa_plan_create_prefix(cfgq, own, pre, shared, T, free)
        for which in (B.ARR_CU_SEQLENS, B.ARR_PAGE_INDPTR, B.ARR_PAGE_INDICES, B.ARR_SLOT_MAPPING, B.ARR_SEQ_LENS,
                      B.ARR_PREFILL_ITEMS, B.ARR_SPLIT_INDPTR, B.ARR_DECODE_ITEMS):
            assert np.array_equal(B.cpa_plan_export(plan, which), B.cpa_plan_export(plain, which)), which
        assert B.cpa_plan_export(plan, B.ARR_SEQ_LENS).tolist() == pre
        B.cpa_plan_destroy(plain)
    finally:
        B.cpa_plan_destroy(plan)
    # errors: the union of the two creators'
    for kw, args in [({}, (own, [0, 200, 512, 768], shared, T, C, free)),           # prefix not whole KV tiles
                     ({}, (own, pre, shared[:10], T, C, free)),                     # prefix longer than the cache
                     ({}, (own, pre, shared, T, 200, free)),                        # chunk not a multiple of 128
                     ({"decode_steps_per_chunk": 0}, (own, pre, shared, T, C, free))]:
        rc, h = B.cpa_plan_create_prefix_chunked(cfg, *args, check=False, **kw)
        assert rc == B.CPA_EINVAL and not h
    rc, h = B.cpa_plan_create_prefix_chunked(cfg, own, pre, shared, T, C, free[:5], check=False)
    assert rc == B.CPA_ENOSPC and not h


def test_event_from_host_argument_checks_and_stage_size():
    cfg = B.cpa_config(8, 2, 128, 16, 0.088, 0, 0, 0)
    lens, T = (300, 50), 3
    plan = B.cpa_plan_create_chunked(cfg, lens, T, 128, np.arange(100, dtype=np.int32))
    tokens, rows = sum(lens), T * len(lens)
    a = lambda n: -(-n // 256) * 256
    want = 2 * a(tokens * 8 * 128 * 2) + 2 * a(tokens * 2 * 128 * 2) + 2 * a(rows * 8 * 128 * 2) + 2 * a(rows * 2 * 128 * 2)
    assert B.cpa_plan_param(plan, B.PARAM_HOST_STAGE_BYTES) == want
    f = 4096
    assert B.cpa_event_host(plan, f, f, f, f, f, f, f, f, f, f, f, f) == B.CPA_ESTATE          # not uploaded
    assert B.cpa_decode_append_steps(plan, f, f, f, f, f, f, f, 2) == B.CPA_ESTATE
    assert B.cpa_decode_append_steps(plan, f, f, f, f, f, f, f, -2) == B.CPA_EINVAL
    assert B.cpa_decode_append_steps(plan, f, f, f, f, f, f, f, 0) == B.CPA_OK
    assert B.cpa_event_host(plan, None, f, f, f, f, f, f, f, f, f, f, f) == B.CPA_EINVAL
    assert B.cpa_event_host(plan, f, f, f, f, None, f, f, f, f, f, f, f) == B.CPA_EINVAL       # T > 0 needs decode inputs
    assert B.cpa_event_host(plan, f, f, f, f, f, f, f, f, f + 16, f, f, f) == B.CPA_EINVAL     # stage not 256-aligned
    B.cpa_plan_destroy(plan)
    dyn = B.cpa_plan_create_dynamic(cfg, lens, T, np.arange(100, dtype=np.int32))
    assert B.cpa_plan_param(dyn, B.PARAM_HOST_STAGE_BYTES) == want
    B.cpa_plan_destroy(dyn)


def test_partition_is_the_papers_rule():
    # Section 4 "Snapshot & partition", Section 5 "Threshold and block size interaction": the printed worker counts,
    # the restated rule on odd sizes, and the creator's error cases
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "worker_counts.txt")) as f:
        rows = [tuple(int(x) for x in line.split()) for line in f if line.strip() and not line.startswith("#")]
    assert rows
    for tau, blk, workers in rows:
        lens = B.cpa_partition(tau, blk)
        assert len(lens) == workers and int(lens.sum()) == tau and (lens[:-1] == blk).all() and 1 <= lens[-1] <= blk
    for tau, blk in [(1, 1), (1, 4096), (4096, 4096), (4097, 4096), (131072, 2048), (100000, 7777)]:
        assert B.cpa_partition(tau, blk).tolist() == op.partition(tau, blk)
    assert B.cpa_partition(0, 16, check=False)[0] == B.CPA_EINVAL
    assert B.cpa_partition(16, 0, check=False)[0] == B.CPA_EINVAL
    assert B.cpa_partition(100, 10, capacity=9, check=False) == (B.CPA_ENOSPC, 10)
    assert B.cpa_partition(1 << 40, 1, capacity=4, check=False)[0] == B.CPA_EUNSUPPORTED


def test_chunked_plan_errors():
    cfg = B.cpa_config(8, 2, 64, 16, 0.125, 0, 0, 0)
    free = np.arange(100, dtype=np.int32)
    for chunk in (0, 64, 200, -128):
        rc, h = B.cpa_plan_create_chunked(cfg, (300, 50), 2, chunk, free, check=False)
        assert rc == B.CPA_EINVAL and not h
    rc, h = B.cpa_plan_create_chunked(cfg, (300, 50), 2, 128, free, decode_sms=4096, check=False)
    assert rc == B.CPA_EINVAL and not h
    rc, h = B.cpa_plan_create_chunked(cfg, (300, 0), 2, 128, free, check=False)
    assert rc == B.CPA_EINVAL and not h
    rc, h = B.cpa_plan_create_chunked(cfg, (300, 50), 2, 128, free, decode_steps_per_chunk=0, check=False)
    assert rc == B.CPA_EINVAL and not h
    fake = 4096
    plan = B.cpa_plan_create_chunked(cfg, (300, 50), 2, 128, free)
    assert B.cpa_step_mixed(plan, 0, fake, fake, fake, fake + 16, fake, fake, fake, fake, fake, fake, fake) == B.CPA_ESTATE  # not uploaded
    B.cpa_plan_destroy(plan)


# ----------------------------------------------------------------------------
# pages on demand: the first assignment
# ----------------------------------------------------------------------------

def test_dynamic_plan_first_assignment_matches_the_model():
    lens = [5, 16, 17, 300, 31, 32]
    T, P = 40, 16
    free = np.random.default_rng(3).permutation(80).astype(np.int32)
    cfg = B.cpa_config(8, 2, 128, P, 0.088, 0, 0, 0)
    plan = B.cpa_plan_create_dynamic(cfg, lens, T, free)
    try:
        m = op.DynamicPages(lens, T, P, free.tolist())
        assert B.cpa_plan_export(plan, B.ARR_PAGES_ASSIGNED).tolist() == m.pages
        indptr, idx = B.cpa_plan_export(plan, B.ARR_PAGE_INDPTR), B.cpa_plan_export(plan, B.ARR_PAGE_INDICES)
        assert np.diff(indptr).tolist() == m.cap                       # a row per block, as long as the block may grow
        assert [idx[indptr[b]:indptr[b] + m.pages[b]].tolist() for b in range(len(lens))] == m.initial
        ring = B.cpa_plan_export(plan, B.ARR_FREE_RING).tolist()
        assert ring == free[sum(m.pages):].tolist()                    # the rest, in free-list order
        assert B.cpa_plan_param(plan, B.PARAM_PAGES_USED) == sum(m.pages)
        # the prefill tokens' slots are those of an ordinary plan over the same first pages
        slots = B.cpa_plan_export(plan, B.ARR_SLOT_MAPPING)
        cu = np.concatenate([[0], np.cumsum(lens)])
        for b, L in enumerate(lens):
            for i in (0, L // 2, L - 1):
                assert slots[cu[b] + i] == m.initial[b][i // P] * P + i % P
        m.check([idx[indptr[b]:indptr[b + 1]].tolist() for b in range(len(lens))], m.pages, lens, ring)
    finally:
        B.cpa_plan_destroy(plan)
    # the free list must cover the first pages; nothing beyond them is needed up front
    need = sum(L // P + 1 for L in lens)
    rc, h = B.cpa_plan_create_dynamic(cfg, lens, T, free[:need - 1], check=False)
    assert rc == B.CPA_ENOSPC and not h
    plan = B.cpa_plan_create_dynamic(cfg, lens, T, free[:need])
    assert len(B.cpa_plan_export(plan, B.ARR_FREE_RING)) == 0
    fake = 4096
    assert B.cpa_decode_append_dynamic(plan, fake, fake, fake, None, fake, fake, fake, fake) == B.CPA_ESTATE   # not uploaded
    assert B.cpa_release_blocks(plan, fake) == B.CPA_ESTATE
    assert B.cpa_plan_sync(plan) == B.CPA_ESTATE
    B.cpa_plan_destroy(plan)


def test_probe_library_is_separate_and_exports_its_entry_point():
    import ctypes
    from paper_2605_23296_b200 import build
    assert os.path.exists(build.PROBE_LIB) and build.PROBE_LIB != B.LIB_PATH
    assert hasattr(ctypes.CDLL(build.PROBE_LIB), "cpa_test_wait_probe")
    assert not hasattr(ctypes.CDLL(B.LIB_PATH), "cpa_test_wait_probe")     # test code stays out of the product


# ----------------------------------------------------------------------------
# prefix-aware layout: shared prefix pages
# ----------------------------------------------------------------------------

def _prefix_plan(w, pages_per_split=0, check=True, prefix_lens=None, shared=None):
    o = w.own
    cfg = B.cpa_config(o.num_q_heads, o.num_kv_heads, o.head_dim, o.page_size, o.scale, 0, pages_per_split, 0)
    return B.cpa_plan_create_prefix(cfg, o.block_lens, w.prefix_lens if prefix_lens is None else prefix_lens,
                                    w.shared_pages if shared is None else shared, o.decode_steps, o.free_pages,
                                    check=check)


@pytest.mark.parametrize("pps", [0, 5])
def test_prefix_plan_bit_exact(pps):
    w = wl.prefix_aware(5, 384, 8, 2, 128, steps=7, seed=3, marker_tokens=21).materialise(with_decode=False)
    o = w.own
    plan = _prefix_plan(w, pps)
    try:
        C = B.cpa_plan_export(plan, B.ARR_SPLIT_PAGES).tolist()
        M = B.cpa_plan_param(plan, B.PARAM_Q_TILE_ROWS)
        CH = B.cpa_plan_param(plan, B.PARAM_SHARED_CHUNK_PAGES)
        assert CH >= 8 and CH % 8 == 0
        ref = op.build_plan(o.block_lens.tolist(), o.decode_steps, o.page_size, o.free_pages.tolist(), o.num_kv_heads,
                            M, C, prefix_lens=w.prefix_lens.tolist(), shared_pages=w.shared_pages.tolist(),
                            shared_chunk_pages=CH)
        even = B.cpa_plan_param(plan, B.PARAM_DECODE_EVEN_CUT)
        for which, key in [(B.ARR_CU_SEQLENS, "cu_seqlens"), (B.ARR_PAGE_INDPTR, "page_indptr"),
                           (B.ARR_PAGE_INDICES, "page_indices"), (B.ARR_SEQ_LENS, "seq_lens"),
                           (B.ARR_SLOT_MAPPING, "slot_mapping"), (B.ARR_PREFILL_ITEMS, "prefill_items"),
                           (B.ARR_DECODE_ITEMS, "decode_items"), (B.ARR_SPLIT_INDPTR, "split_indptr")]:
            if even and key in ("decode_items", "split_indptr"):
                continue
            got = B.cpa_plan_export(plan, which)
            assert np.array_equal(got, np.asarray(ref[key], dtype=np.int32).reshape(got.shape)), key
        own = (-(-(o.block_lens.astype(np.int64) + o.decode_steps) // o.page_size)).tolist()
        check_decode_cut(plan, own, o.num_kv_heads, n_fixed=[-(-(int(x) // o.page_size) // CH) for x in w.prefix_lens])
        ctas = B.cpa_plan_param(plan, B.PARAM_PREFILL_CTAS)
        check_schedule(B.cpa_plan_export(plan, B.ARR_PREFILL_SCHED), ctas, ref["prefill_items"], o.block_lens, M,
                       o.num_q_heads, o.num_kv_heads, prefix_lens=w.prefix_lens)
        assert B.cpa_plan_param(plan, B.PARAM_PAGES_USED) == ref["page_indptr"][-1]
    finally:
        B.cpa_plan_destroy(plan)


def test_prefix_plan_schedule_is_balanced_at_full_size():
    # the paper's layout at bench size: 16 workers x (8192 + 16) own tokens over 15 x 8192 cached ones
    w = wl.prefix_aware(16, 8192, 32, 8, 128, steps=256, seed=11, permute_pages=False)
    o = w.own
    hist_pages = w.hist_tokens // o.page_size
    w.shared_pages = np.arange(hist_pages, dtype=np.int32)
    o.free_pages = np.arange(hist_pages, hist_pages + o.num_pages, dtype=np.int32)
    plan = _prefix_plan(w)
    try:
        items = B.cpa_plan_export(plan, B.ARR_PREFILL_ITEMS).tolist()
        check_schedule(B.cpa_plan_export(plan, B.ARR_PREFILL_SCHED), B.cpa_plan_param(plan, B.PARAM_PREFILL_CTAS), items,
                       o.block_lens, B.cpa_plan_param(plan, B.PARAM_Q_TILE_ROWS), o.num_q_heads, o.num_kv_heads,
                       prefix_lens=w.prefix_lens, balance=1.05)
    finally:
        B.cpa_plan_destroy(plan)


def test_plan_limits_of_packed_fields():
    free = np.arange(100, dtype=np.int32)
    rc, h = B.cpa_plan_create(B.cpa_config(8, 2, 64, 16, 0.125, 0, 0, 4096), (40, 50), 4, free, check=False)
    assert rc == B.CPA_EUNSUPPORTED and not h          # the schedule's keys hold a CTA id in 12 bits
    plan = B.cpa_plan_create(B.cpa_config(8, 2, 64, 16, 0.125, 0, 0, 4095), (40, 50), 4, free)
    B.cpa_plan_destroy(plan)
    # a plan with cached prefixes packs worker ranges in 16 bits
    n = 65536
    cfg = B.cpa_config(8, 2, 64, 16, 0.125, 0, 0, 0)
    rc, h = B.cpa_plan_create_prefix(cfg, np.ones(n, dtype=np.int32), np.zeros(n, dtype=np.int32),
                                     np.zeros(0, dtype=np.int32), 0, np.arange(n, dtype=np.int32), check=False)
    assert rc == B.CPA_EUNSUPPORTED and not h


def test_prefix_plan_errors():
    w = wl.prefix_aware(3, 128, 4, 1, 64, steps=2, seed=1).materialise(with_decode=False)
    for bad in ([0, 128, 200], [0, -128, 256], [0, 128, 16]):       # not a multiple of 128 / negative
        rc, h = _prefix_plan(w, check=False, prefix_lens=bad)
        assert rc == B.CPA_EINVAL and not h
    rc, h = _prefix_plan(w, check=False, shared=w.shared_pages[:-1])  # prefix longer than the shared pages
    assert rc == B.CPA_EINVAL and not h
    w.own.free_pages = w.own.free_pages[:2]                              # own pages do not fit
    rc, h = _prefix_plan(w, check=False)
    assert rc == B.CPA_ENOSPC and not h
