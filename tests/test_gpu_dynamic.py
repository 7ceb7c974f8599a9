"""Pages on demand on the CUDA path (paper, Section 8 "Dynamic block size and prompt selection"; the
many-short-sequences shape of its second benchmark, Section 3.1): summaries stop at different lengths,
nothing is reserved for them, blocks take pages from a common reserve inside the decode launch and give
them back when they have stopped.  Attention must match the oracle's contiguous per-block cache; the
page bookkeeping, where WHICH page a block gets is free, is checked by the oracle model's invariants and
by reading every cached token back from the slot the final page table names."""
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


def _table_rows(s):
    from paper_2605_23296_b200 import binding as B
    indptr, idx = s.export(B.ARR_PAGE_INDPTR), s.export(B.ARR_PAGE_INDICES)
    return [idx[indptr[b]:indptr[b + 1]].tolist() for b in range(len(indptr) - 1)]


def run_dynamic_event(w, stop_lens, spare_pages, release_every=0, what="", prefill_rows=None, check_steps=None):
    """`prefill_rows` / `check_steps`: at full size the oracle sees a sample of the prefill rows and of the decode
    steps (every live block at those steps); the page bookkeeping is checked at every step either way."""
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w.materialise()
    T, Bn, P = w.decode_steps, w.num_blocks, w.page_size
    first = int((w.block_lens // P + 1).sum())
    free = w.free_pages[:first + spare_pages]                 # far fewer pages than B * ceil((L + T) / P)
    assert len(free) < w.pages_needed
    s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, free, w.num_pages, scale=w.scale,
                          poison_pools=True, dynamic_pages=True)
    model = op.DynamicPages(w.block_lens.tolist(), T, P, free.tolist())
    assert s.export(B.ARR_PAGES_ASSIGNED).tolist() == model.pages
    assert len(s.export(B.ARR_FREE_RING)) == model.reserve
    assert [r[:n] for r, n in zip(_table_rows(s), model.pages)] == model.initial

    cu = _cu(w)
    k, v = _dev(w.k), _dev(w.v)
    o = s.prefill(_dev(w.q), k, v)
    if prefill_rows is None:
        assert_attention_close(_bits(o), oa.prefill(w.q, w.k, w.v, cu, w.scale), f"{what} prefill")
    else:
        got = _bits(o[torch.from_numpy(prefill_rows).to("cuda:0")])
        assert_attention_close(got, oa.prefill(w.q, w.k, w.v, cu, w.scale, rows=prefill_rows), f"{what} prefill (sampled rows)")
    s.append_prefill(k, v)
    st = oa.DecodeState(w.k, w.v, cu, T)
    qd, kd, vd = _dev(w.q_dec), _dev(w.k_dec), _dev(w.v_dec)
    released = np.zeros(Bn, dtype=bool)
    for t in range(T):
        active = (t < stop_lens) & ~released
        flags = torch.from_numpy(active.astype(np.int32)).to("cuda:0")
        out = torch.full((Bn, w.num_q_heads, w.head_dim), 5.0, dtype=torch.bfloat16, device="cuda:0")
        s.decode_append_dynamic(qd[t], kd[t], vd[t], flags, out=out)
        model.step(active.tolist())
        live = np.flatnonzero(active).tolist()
        st.append(w.k_dec[t], w.v_dec[t], blocks=live)
        if live and (check_steps is None or t in check_steps):
            want = st.decode(w.q_dec[t], w.scale, blocks=live)
            assert_attention_close(_bits(out)[live], want[live], f"{what} step {t}")
        idle = np.flatnonzero(~active)
        assert (out[torch.from_numpy(idle).to("cuda:0")] == 5.0).all(), f"{what}: step {t} wrote rows of idle blocks"
        if release_every and t % release_every == release_every - 1:
            stopped = (t + 1 >= stop_lens) & ~released
            s.release(torch.from_numpy((~stopped).astype(np.int32)).to("cuda:0"))
            model.release(np.flatnonzero(stopped).tolist())
            released |= stopped
    assert s.status() == 0
    s.sync()
    rows, assigned = _table_rows(s), s.export(B.ARR_PAGES_ASSIGNED).tolist()
    lens = s.export(B.ARR_SEQ_LENS).tolist()
    model.check(rows, assigned, lens, s.export(B.ARR_FREE_RING).tolist())
    # every token of every block that still holds its pages, read back from the slot the final table names
    kp, vp = pool_rows(_bits(s.k_pool)), pool_rows(_bits(s.v_pool))
    for b in range(Bn):
        if released[b]:
            continue
        n = lens[b]
        pages = np.asarray(rows[b])[np.arange(n) // P]
        assert np.array_equal(kp[pages, :, np.arange(n) % P], st.k[b][:n]), f"{what}: K of block {b}"
        assert np.array_equal(vp[pages, :, np.arange(n) % P], st.v[b][:n]), f"{what}: V of block {b}"
    s.close()


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 128), (4, 1, 64)])
def test_summaries_of_different_lengths_without_reserved_pages(hq, hkv, d):
    rng = np.random.default_rng(hq + d)
    lens = rng.integers(40, 200, 24).tolist() + [16, 32, 15, 31]        # some start exactly at a page end
    w = wl.custom(lens, hq, hkv, d, steps=40, seed=91 + d, permute_pages=True)
    stop = rng.integers(5, 41, len(lens)).astype(np.int32)
    run_dynamic_event(w, stop, spare_pages=60, what=f"dynamic {hq}/{hkv}/{d}")


def test_stopped_blocks_give_their_pages_back():
    # the reserve alone (12 pages) could not carry all blocks to the end; the pages of blocks that stop early do
    rng = np.random.default_rng(5)
    lens = rng.integers(30, 120, 20).tolist()
    w = wl.custom(lens, 8, 2, 128, steps=48, seed=93, permute_pages=True)
    stop = np.where(np.arange(20) % 2 == 0, 8, 48).astype(np.int32)      # half of them stop after 8 tokens
    run_dynamic_event(w, stop, spare_pages=12, release_every=8, what="release")


def test_many_short_sequences_at_full_size():
    # the benchmark's second workload as it is timed (192 sequences of 514..1021 tokens, summaries that stop after
    # 33..256 tokens, stopped sequences released every 32 steps): page bookkeeping at every step, the oracle on
    # sampled prefill rows and on every live sequence at sampled steps (page boundaries of the summaries included)
    w = wl.locomo_like().materialise()
    rng = np.random.default_rng(6)
    cu = _cu(w)
    rows = []
    for b, L in enumerate(int(x) for x in w.block_lens):
        cand = {0, 1, 127, 128, 255, 256, 511, 512, L - 2, L - 1} | set(int(x) for x in rng.integers(0, L, 4))
        rows += [cu[b] + r for r in sorted(cand) if 0 <= r < L]
    steps = {0, 1, 15, 16, 17, 31, 32, 33, 63, 64, 127, 128, 200, 254, 255}
    # the pool the benchmark gives it: the first pages plus what the summaries really need (+ 64), not T tokens each
    first = int((w.block_lens // w.page_size + 1).sum())
    need = int((-(-(w.block_lens.astype(np.int64) + w.stop_lens) // w.page_size)).sum())
    run_dynamic_event(w, w.stop_lens, spare_pages=max(first, need) + 64 - first, release_every=32, what="192 short sequences",
                      prefill_rows=np.asarray(rows, dtype=np.int64), check_steps=steps)


def test_whole_batch_without_flags_equals_the_reserved_plan_bitwise():
    # same kernels, same keys per split, other page ids: the outputs are the reserved plan's, bit for bit
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.custom([100, 33, 250, 16], 8, 2, 128, steps=20, seed=94, permute_pages=True).materialise()
    outs = []
    for dyn in (False, True):
        s = CompactionSession(w.block_lens, 20, 8, 2, 128, w.free_pages, w.num_pages, scale=w.scale, poison_pools=True,
                              dynamic_pages=dyn)
        s.append_prefill(_dev(w.k), _dev(w.v))
        res = [_bits(s.decode_append(_dev(w.q_dec[t]), _dev(w.k_dec[t]), _dev(w.v_dec[t]))) for t in range(20)]
        assert s.status() == 0
        outs.append(np.stack(res))
        s.close()
    assert np.array_equal(outs[0], outs[1])


def test_empty_reserve_is_reported_and_nothing_is_written_outside():
    # one spare page for four blocks that all fill a page: the status word says CPA_ENOSPC, the blocks that got no
    # page stop growing, and the poison in every page nobody owns is untouched
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.custom([14, 14, 14, 14], 8, 2, 128, steps=12, seed=95, permute_pages=False).materialise()
    free = w.free_pages[:4 + 1]
    s = CompactionSession(w.block_lens, 12, 8, 2, 128, free, w.num_pages, scale=w.scale, poison_pools=True, dynamic_pages=True)
    s.append_prefill(_dev(w.k), _dev(w.v))
    for t in range(6):
        s.decode_append_dynamic(_dev(w.q_dec[t]), _dev(w.k_dec[t]), _dev(w.v_dec[t]))
    assert s.status() == B.CPA_ENOSPC
    s.sync()
    lens, assigned = s.export(B.ARR_SEQ_LENS).tolist(), s.export(B.ARR_PAGES_ASSIGNED).tolist()
    assert sorted(assigned) == [1, 1, 1, 2] and len(s.export(B.ARR_FREE_RING)) == 0
    assert sorted(lens) == [16, 16, 16, 20]                   # three stopped at their page end, one went on
    nan_bits = _bits(torch.full((1,), float("nan"), dtype=torch.bfloat16))[0]
    kp = _bits(s.k_pool)
    owned = set(free.tolist())
    for page in range(w.num_pages):
        if page not in owned:
            assert (kp[page] == nan_bits).all()
    # a single-token append outside the decode launch takes no pages: refused for this kind of plan
    assert B.cpa_kv_append(s.plan, _dev(w.k_dec[0]), _dev(w.v_dec[0]), None, s.k_pool, s.v_pool) == B.CPA_EUNSUPPORTED
    s.close()
