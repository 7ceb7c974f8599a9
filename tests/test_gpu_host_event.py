"""A whole event from host memory (`cpa_event_host`) against the CPU oracle: the prompts go up chunk by
chunk, every chunk is prefilled when it has landed, outputs come home behind the kernels (paper, Section 4:
each block's prompt is prefilled and its summary decoded).  Same results as the device-side calls: prefill
rows and decode tokens within tolerance of the oracle, pools bit for bit."""
import numpy as np
import pytest

from _util import assert_attention_close, pool_rows
from oracle import attention as oa
from oracle import plan as op
from paper_2605_23296_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _pinned(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).pin_memory()


def _host_bits(t):
    import torch
    return t.view(torch.int16).numpy().view(np.uint16)


def _dev_bits(t):
    from paper_2605_23296_b200.session import tensor_to_bits
    return tensor_to_bits(t)


def run_host_event(w, chunk, what, pageable=False, twice=False):
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w.materialise()
    T, Bn = w.decode_steps, w.num_blocks
    s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages, w.num_pages,
                          scale=w.scale, poison_pools=True, chunk_tokens=chunk, decode_sms=1 if chunk else 0)
    mk = (lambda b: torch.from_numpy(b.view(np.int16).copy()).view(torch.bfloat16)) if pageable else _pinned
    h_q, h_k, h_v = mk(w.q), mk(w.k), mk(w.v)
    h_o = torch.full(h_q.shape, 7.0, dtype=torch.bfloat16)
    h_o = h_o if pageable else h_o.pin_memory()
    if T:
        h_qd, h_kd, h_vd = mk(w.q_dec), mk(w.k_dec), mk(w.v_dec)
        h_od = torch.full(h_qd.shape, 5.0, dtype=torch.bfloat16)
        h_od = h_od if pageable else h_od.pin_memory()
    else:
        h_qd = h_kd = h_vd = h_od = None
    stage = s.event_from_host(h_q, h_k, h_v, h_o, h_qd, h_kd, h_vd, h_od)
    torch.cuda.synchronize()
    assert s.status() == 0
    if twice:
        # the plan is used up until it is uploaded again
        assert B.cpa_event_host(s.plan, h_q, h_k, h_v, h_o, h_qd, h_kd, h_vd, h_od, stage, s.k_pool, s.v_pool,
                                s.workspace) == B.CPA_ESTATE
    cu = np.concatenate([[0], np.cumsum(w.block_lens.astype(np.int64))])
    assert_attention_close(_host_bits(h_o), oa.prefill(w.q, w.k, w.v, cu, w.scale), f"{what} prefill from host")
    state = oa.DecodeState(w.k, w.v, cu, T)
    for t in range(T):
        state.append(w.k_dec[t], w.v_dec[t])
        assert_attention_close(_host_bits(h_od[t]), state.decode(w.q_dec[t], w.scale), f"{what} decode step {t}")
    plan = op.build_plan(w.block_lens.tolist(), T, w.page_size, w.free_pages.tolist(), w.num_kv_heads, 128, 1)
    slots = list(plan["slot_mapping"])
    ks, vs = [w.k], [w.v]
    for t in range(T):
        slots += [op.slot_of(plan, w.page_size, b, int(w.block_lens[b]) + t) for b in range(Bn)]
        ks.append(w.k_dec[t])
        vs.append(w.v_dec[t])
    kp, vp, written = oa.expected_pool(slots, np.concatenate(ks), np.concatenate(vs), w.num_pages, w.page_size)
    mask = np.broadcast_to(written[:, None, :, None], kp.shape)
    assert np.array_equal(pool_rows(_dev_bits(s.k_pool))[mask], kp[mask])
    assert np.array_equal(pool_rows(_dev_bits(s.v_pool))[mask], vp[mask])
    assert np.array_equal(s.export(B.ARR_SEQ_LENS), w.block_lens + T)
    s.sync()
    assert np.array_equal(s.export(B.ARR_SEQ_LENS), w.block_lens + T)     # the device's own lengths
    s.close()


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 128), (4, 1, 64)])
def test_chunks_go_up_one_by_one(hq, hkv, d):
    run_host_event(wl.custom([700, 130, 50, 513], hq, hkv, d, steps=4, seed=100 + d), 256, f"chunked {hq}/{hkv}/{d}", twice=True)


def test_plan_without_chunks_runs_the_same_steps_unpipelined():
    run_host_event(wl.custom([300, 100, 129], 8, 2, 128, steps=3, seed=103), 0, "whole blocks")


def test_pageable_host_memory_is_slower_not_wrong():
    run_host_event(wl.custom([300, 100, 129], 8, 2, 128, steps=2, seed=104), 128, "pageable", pageable=True)


def test_no_decode_steps_and_null_decode_buffers():
    run_host_event(wl.custom([400, 130], 8, 2, 128, steps=0, seed=105), 128, "T = 0")


def test_a_second_event_reuses_stage_and_streams_after_a_new_upload():
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.custom([600, 200], 8, 2, 128, steps=2, seed=106).materialise()
    s = CompactionSession(w.block_lens, 2, 8, 2, 128, w.free_pages, w.num_pages, scale=w.scale, chunk_tokens=256, decode_sms=1)
    h = [_pinned(x) for x in (w.q, w.k, w.v, w.q_dec, w.k_dec, w.v_dec)]
    outs = []
    stage = None
    for i in range(2):
        h_o, h_od = torch.zeros_like(h[0]).pin_memory(), torch.zeros_like(h[3]).pin_memory()
        stage = s.event_from_host(h[0], h[1], h[2], h_o, h[3], h[4], h[5], h_od, stage=stage)
        torch.cuda.synchronize()
        assert s.status() == 0
        outs.append((_host_bits(h_o).copy(), _host_bits(h_od).copy()))
        if i == 0:
            nbytes = s.param(B.PARAM_INDEX_BYTES)
            s._check(B.cpa_plan_upload(s.plan, s.index_buf, nbytes, s._stream()), "cpa_plan_upload")
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    s.close()


@pytest.mark.parametrize("chunk", [256, 0])
def test_prefix_aware_workers_from_host(chunk):
    # both layouts' planner paths in one event: history cached first, workers' own tokens from the host, in chunks
    # or (chunk 0: a plain prefix-aware plan) whole
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor
    w = wl.prefix_aware(3, 256, 8, 2, 128, steps=3, seed=107, own_lens=[272, 600, 129]).materialise()
    o = w.own
    shape = (w.num_pages, o.num_kv_heads, o.page_size, o.head_dim)
    pools = (torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda:0"),
             torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda:0"))
    hist = CompactionSession([w.hist_tokens], 0, o.num_q_heads, o.num_kv_heads, o.head_dim, w.shared_pages,
                             w.num_pages, scale=o.scale, pools=pools)
    hist.append_prefill(bits_to_tensor(w.k_hist, "cuda:0"), bits_to_tensor(w.v_hist, "cuda:0"))
    s = CompactionSession(o.block_lens, o.decode_steps, o.num_q_heads, o.num_kv_heads, o.head_dim, o.free_pages,
                          w.num_pages, scale=o.scale, prefix_lens=w.prefix_lens, shared_pages=w.shared_pages,
                          pools=pools, chunk_tokens=chunk, decode_sms=1 if chunk else 0)
    h = [_pinned(x) for x in (o.q, o.k, o.v, o.q_dec, o.k_dec, o.v_dec)]
    h_o, h_od = torch.zeros_like(h[0]).pin_memory(), torch.zeros_like(h[3]).pin_memory()
    s.event_from_host(h[0], h[1], h[2], h_o, h[3], h[4], h[5], h_od)
    torch.cuda.synchronize()
    assert s.status() == 0
    cu = np.concatenate([[0], np.cumsum(o.block_lens.astype(np.int64))])
    assert_attention_close(_host_bits(h_o), oa.prefill_prefix_aware(o.q, o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.scale),
                           "prefix-aware prefill from host")
    st = oa.PrefixDecodeState(o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.decode_steps)
    for t in range(o.decode_steps):
        st.append(o.k_dec[t], o.v_dec[t])
        assert_attention_close(_host_bits(h_od[t]), st.decode(o.q_dec[t], o.scale), f"prefix-aware decode step {t} from host")
    assert np.array_equal(s.export(B.ARR_SEQ_LENS), w.prefix_lens + o.block_lens + o.decode_steps)
    s.close()
    hist.close()


def test_ragged_at_full_size_through_the_host_call():
    # the benchmark's end-to-end leg as it is timed: the default workload, chunks of 4096 tokens, pinned host
    # buffers; prefill on sampled rows (block ends, tile and chunk boundaries, random rows), every block and head of
    # the decode at sampled steps, lengths at the end
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession
    w = wl.ragged().materialise()
    T, chunk = w.decode_steps, 4096
    s = CompactionSession(w.block_lens, T, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages, w.num_pages,
                          scale=w.scale, chunk_tokens=chunk, decode_sms=1)
    h = [_pinned(x) for x in (w.q, w.k, w.v, w.q_dec, w.k_dec, w.v_dec)]
    h_o = torch.empty(h[0].shape, dtype=torch.bfloat16).pin_memory()
    h_od = torch.empty(h[3].shape, dtype=torch.bfloat16).pin_memory()
    s.event_from_host(h[0], h[1], h[2], h_o, h[3], h[4], h[5], h_od)
    torch.cuda.synchronize()
    assert s.status() == 0
    cu = np.concatenate([[0], np.cumsum(w.block_lens.astype(np.int64))])
    rng = np.random.default_rng(2)
    rows = []
    for b, L in enumerate(int(x) for x in w.block_lens):
        cand = {0, 1, 127, 128, L - 2, L - 1} | {c + d for c in range(chunk, L, chunk) for d in (-1, 0, 1)}
        cand |= set(int(x) for x in rng.integers(0, L, 4))
        rows += [cu[b] + r for r in sorted(cand) if 0 <= r < L]
    rows = np.asarray(rows, dtype=np.int64)
    assert_attention_close(_host_bits(h_o)[rows], oa.prefill(w.q, w.k, w.v, cu, w.scale, rows=rows),
                           "ragged prefill from host (sampled rows)", allow_big=False)
    checks = {0, 1, 15, 16, 17, 300, T - 1}
    st = oa.DecodeState(w.k, w.v, cu, T)
    for t in range(T):
        st.append(w.k_dec[t], w.v_dec[t])
        if t in checks:
            assert_attention_close(_host_bits(h_od[t]), st.decode(w.q_dec[t], w.scale), f"ragged decode step {t} from host",
                                   allow_big=False)
    assert np.array_equal(s.export(B.ARR_SEQ_LENS), w.block_lens + T)
    s.close()
