"""Asynchronous compaction (paper, Section 8 "Discussion and Future Work": run the compaction workers in
the background while the agent continues) as far as attention goes: an event runs on whatever stream
the caller gives it, inside an SM budget (`cpa_config.num_sms`).  A reduced budget changes the launch
shapes -- a short persistent prefill grid whose CTAs walk more units each, a decode wave smaller than
the item list so that CTAs loop over items -- and must not change the results; and two events on two
streams of different priority must both match the oracle."""
import numpy as np
import pytest

from _util import assert_attention_close
from oracle import attention as oa
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


def _event(w, num_sms, fused=True):
    """One whole event with an SM budget; returns (session, prefill output bits, [decode output bits])."""
    from paper_2605_23296_b200.session import CompactionSession
    s = CompactionSession(w.block_lens, w.decode_steps, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages,
                          w.num_pages, scale=w.scale, poison_pools=True, num_sms=num_sms)
    k, v = _dev(w.k), _dev(w.v)
    o = s.prefill(_dev(w.q), k, v)
    s.append_prefill(k, v)
    outs = []
    for t in range(w.decode_steps):
        if fused:
            outs.append(s.decode_append(_dev(w.q_dec[t]), _dev(w.k_dec[t]), _dev(w.v_dec[t])))
        else:
            s.append(_dev(w.k_dec[t]), _dev(w.v_dec[t]))
            outs.append(s.decode(_dev(w.q_dec[t])))
    return s, o, outs


def _check(w, o, outs, what):
    assert_attention_close(_bits(o), oa.prefill(w.q, w.k, w.v, _cu(w), w.scale), f"{what} prefill")
    st = oa.DecodeState(w.k, w.v, _cu(w), w.decode_steps)
    for t in range(w.decode_steps):
        st.append(w.k_dec[t], w.v_dec[t])
        assert_attention_close(_bits(outs[t]), st.decode(w.q_dec[t], w.scale), f"{what} decode step {t}")


@pytest.mark.parametrize("num_sms", [16, 37, 74])
def test_dense_shape_with_an_sm_budget(num_sms):
    from paper_2605_23296_b200 import binding as B
    w = wl.custom([1024] * 8, 32, 8, 128, steps=6, seed=61, permute_pages=False).materialise()   # the 8B shape, shrunk
    s, o, outs = _event(w, num_sms)
    assert s.status() == 0
    assert s.param(B.PARAM_PREFILL_CTAS) == num_sms                 # a short persistent grid: 8 x 4 x 32 units on it
    n_items = s.export(B.ARR_DECODE_ITEMS).shape[0]
    if num_sms == 16:
        assert n_items > 3 * num_sms                                 # more items than the wave holds: CTAs loop
    _check(w, o, outs, f"dense shape, {num_sms} SMs")
    s.close()


@pytest.mark.parametrize("num_sms,fused", [(37, True), (74, False)])
def test_ragged_shape_with_an_sm_budget(num_sms, fused):
    from paper_2605_23296_b200 import binding as B
    w = wl.ragged(seed=62, num_blocks=32, lo=100, hi=900, steps=5).materialise()   # 32 x 8 (block, kv head) pairs
    s, o, outs = _event(w, num_sms, fused=fused)
    assert s.status() == 0
    n_items = s.export(B.ARR_DECODE_ITEMS).shape[0]
    assert n_items >= 256 and (num_sms != 37 or n_items > 3 * num_sms)
    _check(w, o, outs, f"ragged shape, {num_sms} SMs")
    s.close()


def test_two_events_on_two_streams_of_different_priority():
    # a background event with half the SMs on a low-priority stream, a foreground event on a high-priority
    # one, their calls interleaved on the host: both results are the oracle's
    import torch
    dev = torch.device("cuda:0")
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    lo_prio, hi_prio = torch.cuda.Stream(dev, priority=0), torch.cuda.Stream(dev, priority=-1)
    wb = wl.custom([1536] * 6, 32, 8, 128, steps=4, seed=63).materialise()
    wf = wl.custom([3000, 700], 32, 8, 128, steps=4, seed=64).materialise()
    from paper_2605_23296_b200.session import CompactionSession
    res = {}
    with torch.cuda.stream(lo_prio):
        sb = CompactionSession(wb.block_lens, wb.decode_steps, wb.num_q_heads, wb.num_kv_heads, wb.head_dim,
                               wb.free_pages, wb.num_pages, scale=wb.scale, num_sms=sms // 2)
        kb, vb = _dev(wb.k), _dev(wb.v)
        qb, qdb, kdb, vdb = _dev(wb.q), _dev(wb.q_dec), _dev(wb.k_dec), _dev(wb.v_dec)
    with torch.cuda.stream(hi_prio):
        sf = CompactionSession(wf.block_lens, wf.decode_steps, wf.num_q_heads, wf.num_kv_heads, wf.head_dim,
                               wf.free_pages, wf.num_pages, scale=wf.scale)
        kf, vf = _dev(wf.k), _dev(wf.v)
        qf, qdf, kdf, vdf = _dev(wf.q), _dev(wf.q_dec), _dev(wf.k_dec), _dev(wf.v_dec)
    torch.cuda.synchronize(dev)
    with torch.cuda.stream(lo_prio):
        res["ob"] = sb.prefill(qb, kb, vb)
        sb.append_prefill(kb, vb)
    with torch.cuda.stream(hi_prio):
        res["of"] = sf.prefill(qf, kf, vf)
        sf.append_prefill(kf, vf)
    outs_b, outs_f = [], []
    for t in range(4):
        with torch.cuda.stream(lo_prio):
            outs_b.append(sb.decode_append(qdb[t], kdb[t], vdb[t]))
        with torch.cuda.stream(hi_prio):
            outs_f.append(sf.decode_append(qdf[t], kdf[t], vdf[t]))
    torch.cuda.synchronize(dev)
    with torch.cuda.stream(lo_prio):
        assert sb.status() == 0
    with torch.cuda.stream(hi_prio):
        assert sf.status() == 0
    _check(wb, res["ob"], outs_b, "background event")
    _check(wf, res["of"], outs_f, "foreground event")
    sb.close()
    sf.close()
