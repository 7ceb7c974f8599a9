"""Chunked prefill and mixed steps on the CUDA path against the CPU oracle (paper, Section 4.2: the
serving engine runs with chunked prefill enabled; Section 6: 16k blocks are prefill-bound).  Every step
prefills the next chunk of the blocks that have one and decodes one token of the blocks whose turn it
is; the prefill rows must be the rows of the unchunked prefill, the decode outputs those of the
per-block contiguous cache, the pools bit-exact."""
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


def _cu(w):
    return np.concatenate([[0], np.cumsum(w.block_lens.astype(np.int64))])


def run_chunked_event(w, chunk, decode_sms=0, rows=None, what="", r=1, sparse_pool=False):
    """All steps of the schedule through cpa_step_mixed.  Inputs of decode step t of a block are row t of
    w.*_dec (so a block's t-th summary token has the same inputs whatever step it is produced in)."""
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w.materialise()
    T, Bn = w.decode_steps, w.num_blocks
    s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages, w.num_pages,
                          scale=w.scale, poison_pools=not sparse_pool, chunk_tokens=chunk, decode_sms=decode_sms,
                          decode_steps_per_chunk=r)
    sched = op.mixed_schedule(w.block_lens.tolist(), chunk, T, r)
    assert s.param(B.PARAM_NUM_STEPS) == len(sched)
    start = s.export(B.ARR_DEC_START)
    q, k, v = _dev(w.q), _dev(w.k), _dev(w.v)
    o = torch.full_like(q, 7.0)
    qd, kd, vd = (_dev(w.q_dec), _dev(w.k_dec), _dev(w.v_dec)) if T else (None, None, None)
    dec_out = {}
    cu = _cu(w)
    for step, st in enumerate(sched):
        # this step's decode inputs: block b is at its token t = step - start[b]
        act = st["decode"]
        q_in = torch.zeros((Bn, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device="cuda:0")
        k_in = torch.zeros((Bn, w.num_kv_heads, w.head_dim), dtype=torch.bfloat16, device="cuda:0")
        v_in = torch.zeros_like(k_in)
        for b in act:
            t = step - int(start[b])
            q_in[b], k_in[b], v_in[b] = qd[t, b], kd[t, b], vd[t, b]
        out = torch.full_like(q_in, 5.0)
        s.step_mixed(step, q, k, v, o, q_in, k_in, v_in, out)
        got = _bits(out)
        for b in range(Bn):
            if b in act:
                dec_out[(step, b)] = got[b]
            else:
                assert (out[b] == 5.0).all(), f"{what}: step {step} wrote the output row of idle block {b}"
    assert s.status() == 0
    from paper_2605_23296_b200 import binding as B2
    # out of order: the schedule is over
    assert B2.cpa_step_mixed(s.plan, 0, q, k, v, o, q_in, k_in, v_in, out, s.k_pool, s.v_pool, s.workspace) == B2.CPA_ESTATE

    # ---- prefill rows = the rows of the unchunked prefill
    if rows is None:
        assert_attention_close(_bits(o), oa.prefill(w.q, w.k, w.v, cu, w.scale), f"{what} chunked prefill")
    else:
        got = _bits(o[torch.from_numpy(rows).to("cuda:0")])
        assert_attention_close(got, oa.prefill(w.q, w.k, w.v, cu, w.scale, rows=rows), f"{what} chunked prefill (sampled rows)")
    # ---- decode: block b's token t over its contiguous cache
    state = oa.DecodeState(w.k, w.v, cu, T)
    for t in range(T):
        state.append(w.k_dec[t], w.v_dec[t])
        want = state.decode(w.q_dec[t], w.scale)
        for b in range(Bn):
            assert_attention_close(dec_out[(int(start[b]) + t, b)], want[b], f"{what} block {b} token {t}")
    # ---- pools: every token in its slot, bit for bit; lengths
    plan = op.build_plan(w.block_lens.tolist(), T, w.page_size, w.free_pages.tolist(), w.num_kv_heads, 128, 1)
    slots = list(plan["slot_mapping"])
    ks, vs = [w.k], [w.v]
    for t in range(T):
        slots += [op.slot_of(plan, w.page_size, b, int(w.block_lens[b]) + t) for b in range(Bn)]
        ks.append(w.k_dec[t])
        vs.append(w.v_dec[t])
    if sparse_pool:
        # a pool of many gigabytes with a few pages in use: compare the written slots only, page by page
        k_all, v_all = np.concatenate(ks), np.concatenate(vs)
        for pool, want in ((s.k_pool, k_all), (s.v_pool, v_all)):
            pages = {}
            for i, slot in enumerate(slots):
                page, off = slot // w.page_size, slot % w.page_size
                if page not in pages:
                    pages[page] = pool_rows(_bits(pool[page:page + 1]))[0]
                assert np.array_equal(pages[page][:, off], want[i]), (i, slot)
    elif T or rows is None:
        kp, vp, written = oa.expected_pool(slots, np.concatenate(ks), np.concatenate(vs), w.num_pages, w.page_size)
        mask = np.broadcast_to(written[:, None, :, None], kp.shape)
        assert np.array_equal(pool_rows(_bits(s.k_pool))[mask], kp[mask])
        assert np.array_equal(pool_rows(_bits(s.v_pool))[mask], vp[mask])
    assert np.array_equal(s.export(B.ARR_SEQ_LENS), w.block_lens + T)
    s.close()


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (8, 2, 128), (4, 4, 128)])
def test_chunks_of_one_tile(hq, hkv, d):
    # the hand-worked shape plus a block that ends one token into its second chunk
    run_chunked_event(wl.custom([300, 100, 50, 129], hq, hkv, d, steps=3, seed=hq + d), 128, what=f"chunk 128 {hq}/{hkv}/{d}")


def test_chunks_of_three_tiles_and_a_small_decode_share():
    # 384-token chunks: a 256-row item and a 128-row item per chunk; one SM for the decode wave
    run_chunked_event(wl.custom([1000, 400, 385, 7], 8, 2, 128, steps=4, seed=77), 384, decode_sms=1, what="chunk 384")


@pytest.mark.parametrize("r", [2, 5])
def test_several_decode_steps_beside_one_chunk(r):
    # the short blocks finish their summaries (6 tokens) while the long block is still on its second and third
    # chunk, sit out until the schedule ends, and the long block starts to decode right after its last chunk
    run_chunked_event(wl.custom([700, 100, 50, 129], 8, 2, 128, steps=6, seed=80 + r), 256, what=f"r = {r}", r=r)


def test_page_ids_on_both_sides_of_the_four_gigabyte_line():
    # 8 kv heads x 16 tokens x 128 dims x 2 bytes = 32 KiB per page and pool: page 131072 starts at byte 2^32.  The
    # blocks' pages come from just below and well above that line, in a seeded shuffle, so every path that turns a
    # page id into an address (chunk append, cached-prefix tiles of later chunks through tensor maps, decode's bulk
    # copies, the fused append) has to do it in 64 bits.  The pools (9.2 GB together) are left uninitialised.
    w = wl.custom([700, 130, 385], 32, 8, 128, steps=3, seed=111).materialise()
    n = w.pages_needed
    ids = np.concatenate([np.arange(131072 - n // 2, 131072), np.arange(147000, 147000 + n - n // 2)])
    w.free_pages = np.random.default_rng(111).permutation(ids).astype(np.int32)
    w.spare_pages = int(ids.max()) + 1 - n
    assert w.num_pages * 32768 > 2 ** 32
    run_chunked_event(w, 256, what="pages beyond 4 GB", r=2, sparse_pool=True)


def test_one_chunk_covers_every_block():
    # chunk longer than every block: step 0 is the whole prefill, then plain decode steps
    run_chunked_event(wl.tiny(4), 512, what="tiny, one chunk")


def test_no_decode_steps():
    run_chunked_event(wl.custom([700, 130], 8, 2, 128, steps=0, seed=78), 256, what="T = 0")


def test_long_block_beside_short_ones_sampled_rows():
    # the case chunking is for: a 16k block next to four 2k blocks (8B-class heads), 2048-token chunks;
    # the short blocks decode while the long one is still prefilling
    w = wl.custom([16384, 2048, 2048, 2048, 2048], 32, 8, 128, steps=10, seed=79, permute_pages=True).materialise()
    rng = np.random.default_rng(79)
    cu = _cu(w)
    rows = []
    for b, L in enumerate(int(x) for x in w.block_lens):
        cand = {0, 1, L - 1} | {c for t in range(2048, L, 2048) for c in (t - 1, t, t + 1)} | set(int(x) for x in rng.integers(0, L, 10))
        rows += [cu[b] + r for r in sorted(cand) if 0 <= r < L]
    run_chunked_event(w, 2048, rows=np.asarray(rows, dtype=np.int64), what="16k + 4 x 2k", r=3)


def run_prefix_chunked_event(w, chunk, r=1, decode_sms=0, what=""):
    """The prefix-aware layout with chunked prefill (Section 4.2: prefix caching and chunked prefill both on):
    the history is cached first through a plan of its own; worker b then runs its own tokens chunk by chunk
    over history prefix + earlier chunks, and decodes over prefix + own tokens + its summary so far."""
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w.materialise()
    o = w.own
    T, Bn, P = o.decode_steps, o.num_blocks, o.page_size
    shape = (w.num_pages, o.num_kv_heads, P, o.head_dim)
    pools = (torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda:0"),
             torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda:0"))
    hist = CompactionSession([w.hist_tokens], 0, o.num_q_heads, o.num_kv_heads, o.head_dim, w.shared_pages,
                             w.num_pages, scale=o.scale, pools=pools)
    hist.append_prefill(_dev(w.k_hist), _dev(w.v_hist))
    s = CompactionSession(o.block_lens, T, o.num_q_heads, o.num_kv_heads, o.head_dim, o.free_pages, w.num_pages,
                          scale=o.scale, prefix_lens=w.prefix_lens, shared_pages=w.shared_pages, pools=pools,
                          chunk_tokens=chunk, decode_sms=decode_sms, decode_steps_per_chunk=r)
    sched = op.mixed_schedule(o.block_lens.tolist(), chunk, T, r)    # the schedule does not depend on the prefix
    assert s.param(B.PARAM_NUM_STEPS) == len(sched)
    start = s.export(B.ARR_DEC_START)
    q, k, v = _dev(o.q), _dev(o.k), _dev(o.v)
    out_pre = torch.full_like(q, 7.0)
    qd, kd, vd = _dev(o.q_dec), _dev(o.k_dec), _dev(o.v_dec)
    dec_out = {}
    cu = np.concatenate([[0], np.cumsum(o.block_lens.astype(np.int64))])
    for step, st in enumerate(sched):
        act = st["decode"]
        q_in = torch.zeros((Bn, o.num_q_heads, o.head_dim), dtype=torch.bfloat16, device="cuda:0")
        k_in = torch.zeros((Bn, o.num_kv_heads, o.head_dim), dtype=torch.bfloat16, device="cuda:0")
        v_in = torch.zeros_like(k_in)
        for b in act:
            t = step - int(start[b])
            q_in[b], k_in[b], v_in[b] = qd[t, b], kd[t, b], vd[t, b]
        out = torch.full_like(q_in, 5.0)
        s.step_mixed(step, q, k, v, out_pre, q_in, k_in, v_in, out)
        got = _bits(out)
        for b in range(Bn):
            if b in act:
                dec_out[(step, b)] = got[b]
            else:
                assert (out[b] == 5.0).all(), f"{what}: step {step} wrote the output row of idle worker {b}"
    assert s.status() == 0
    # ---- prefill rows: those of the unchunked prefix-aware prefill; one chunk also by its own definition
    got_pre = _bits(out_pre)
    assert_attention_close(got_pre, oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale),
                           f"{what} chunked prefix-aware prefill")
    wk = Bn - 1
    first = (int(o.block_lens[wk]) - 1) // chunk * chunk        # the worker's last chunk
    n = int(o.block_lens[wk]) - first
    want = oa.prefill_chunk_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale, wk, first, n)
    assert_attention_close(got_pre[cu[wk] + first: cu[wk] + first + n], want, f"{what} last chunk of worker {wk}")
    # ---- decode over shared prefix pages + own pages
    state = oa.PrefixDecodeState(o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, T)
    for t in range(T):
        state.append(o.k_dec[t], o.v_dec[t])
        want = state.decode(o.q_dec[t], o.scale)
        for b in range(Bn):
            assert_attention_close(dec_out[(int(start[b]) + t, b)], want[b], f"{what} worker {b} token {t}")
    # ---- pools: own tokens and summary tokens behind the prefix, the history untouched, bit for bit
    ref = op.build_plan(o.block_lens.tolist(), T, P, o.free_pages.tolist(), o.num_kv_heads, 128, 1,
                        prefix_lens=w.prefix_lens.tolist(), shared_pages=w.shared_pages.tolist(), shared_chunk_pages=16)
    assert np.array_equal(s.export(B.ARR_PAGE_INDICES), np.asarray(ref["page_indices"], dtype=np.int32))
    kp, vp = pool_rows(_bits(s.k_pool)), pool_rows(_bits(s.v_pool))
    for i, slot in enumerate(ref["slot_mapping"]):
        assert np.array_equal(kp[slot // P, :, slot % P], o.k[i]) and np.array_equal(vp[slot // P, :, slot % P], o.v[i])
    for t in range(T):
        for b in range(Bn):
            slot = op.slot_of(ref, P, b, int(w.prefix_lens[b]) + int(o.block_lens[b]) + t)
            assert np.array_equal(kp[slot // P, :, slot % P], o.k_dec[t][b])
            assert np.array_equal(vp[slot // P, :, slot % P], o.v_dec[t][b])
    for t in range(w.hist_tokens):
        page = int(w.shared_pages[t // P])
        assert np.array_equal(kp[page, :, t % P], w.k_hist[t]) and np.array_equal(vp[page, :, t % P], w.v_hist[t])
    assert np.array_equal(s.export(B.ARR_SEQ_LENS), w.prefix_lens + o.block_lens + T)
    s.close()
    hist.close()


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 128), (4, 1, 64)])
def test_prefix_aware_workers_in_chunks(hq, hkv, d):
    # four workers over a history of 256-token blocks; own lengths from one tile to three chunks, ragged ends
    w = wl.prefix_aware(4, 256, hq, hkv, d, steps=4, seed=90 + d, own_lens=[272, 700, 129, 50])
    run_prefix_chunked_event(w, 256, r=2, what=f"prefix + chunks {hq}/{hkv}/{d}")


def test_prefix_aware_chunks_of_one_tile_with_one_decode_sm():
    w = wl.prefix_aware(3, 384, 8, 8, 128, steps=3, seed=93, own_lens=[400, 130, 385])
    run_prefix_chunked_event(w, 128, r=1, decode_sms=1, what="prefix + 128-token chunks")


def test_a_range_of_steps_in_one_call_is_the_single_steps():
    # cpa_step_mixed_range is cpa_step_mixed in a loop inside the library: outputs, pools and lengths bit for bit
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.custom([700, 100, 50, 129], 8, 2, 128, steps=5, seed=97).materialise()
    T, Bn = 5, 4
    q, k, v = _dev(w.q), _dev(w.k), _dev(w.v)
    qd, kd, vd = _dev(w.q_dec), _dev(w.k_dec), _dev(w.v_dec)
    res = []
    for ranged in (False, True):
        s = CompactionSession(w.block_lens, T, 8, 2, 128, w.free_pages, w.num_pages, scale=w.scale, poison_pools=True,
                              chunk_tokens=256, decode_steps_per_chunk=2)
        n = s.param(B.PARAM_NUM_STEPS)
        start = torch.from_numpy(s.export(B.ARR_DEC_START).astype(np.int64)).to("cuda:0")
        ar = torch.arange(Bn, device="cuda:0")
        t_of = [torch.clamp(step - start, 0, T - 1) for step in range(n)]
        q_in = torch.stack([qd[t, ar] for t in t_of]).contiguous()
        k_in = torch.stack([kd[t, ar] for t in t_of]).contiguous()
        v_in = torch.stack([vd[t, ar] for t in t_of]).contiguous()
        o = torch.zeros_like(q)
        out = torch.full_like(q_in, 5.0)
        if ranged:
            s.step_mixed_range(0, 3, q, k, v, o, q_in[:3], k_in[:3], v_in[:3], out[:3])
            s.step_mixed_range(3, n - 3, q, k, v, o, q_in[3:], k_in[3:], v_in[3:], out[3:])
        else:
            for step in range(n):
                s.step_mixed(step, q, k, v, o, q_in[step], k_in[step], v_in[step], out[step])
        assert s.status() == 0
        res.append((_bits(o), _bits(out), _bits(s.k_pool), _bits(s.v_pool), s.export(B.ARR_SEQ_LENS).copy()))
        s.close()
    for a, b in zip(res[0], res[1]):
        assert np.array_equal(a, b)


def test_mixed_step_needs_a_chunked_plan():
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.tiny(2).materialise()
    s = CompactionSession(w.block_lens, 2, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages, w.num_pages)
    q = _dev(w.q)
    assert B.cpa_step_mixed(s.plan, 0, q, q, q, q, None, None, None, None, s.k_pool, s.v_pool, s.workspace) == B.CPA_ESTATE
    s.close()
