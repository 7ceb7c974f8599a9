"""cpa_decode_static: the decode entry point for callers that cannot provide scratch memory
(for instance a plugin limited to the buffers its host framework gave it, or a service whose
device memory was budgeted in full at start-up).  Its split partials live in a fixed array
inside the library.  It runs the same kernels as cpa_decode on the same inputs, so its output
must be cpa_decode's bit for bit, call after call, although the array keeps old contents; and
both must match the CPU oracle.

Collected last on purpose: a run that stops at the first failure has then already run
every other test."""
import numpy as np
import pytest

from _util import assert_attention_close
from oracle import attention as oa
from paper_2605_23296_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_and_oracle_twice():
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor, tensor_to_bits

    w = wl.custom([700, 33, 257, 1200], 8, 2, 128, steps=3, seed=41).materialise()
    s = CompactionSession(w.block_lens, w.decode_steps, w.num_q_heads, w.num_kv_heads, w.head_dim,
                          w.free_pages, w.num_pages, scale=w.scale, poison_pools=True)
    assert s.param(B.PARAM_DECODE_WORKSPACE_BYTES) <= B.STATIC_SCRATCH_BYTES
    assert s.param(B.PARAM_TOTAL_SPLITS) > w.num_blocks          # there are partials to merge
    dev = lambda a: bits_to_tensor(a, "cuda:0")
    s.append_prefill(dev(w.k), dev(w.v))
    cu = np.concatenate([[0], np.cumsum(w.block_lens.astype(np.int64))])
    st = oa.DecodeState(w.k, w.v, cu, w.decode_steps)
    stream = int(torch.cuda.current_stream().cuda_stream)
    for t in range(2):          # two calls in a row: the second one finds the first one's partials
        s.append(dev(w.k_dec[t]), dev(w.v_dec[t]))
        st.append(w.k_dec[t], w.v_dec[t])
        q = dev(w.q_dec[t])
        want = s.decode(q)
        got = torch.full_like(want, 9.0)
        rc = B.cpa_decode_static(s.plan, q, s.k_pool, s.v_pool, got, stream)
        assert rc == B.CPA_OK, B.cpa_strerror(rc)
        assert s.status() == 0
        assert np.array_equal(tensor_to_bits(got), tensor_to_bits(want)), f"call {t}: differs from cpa_decode"
        assert_attention_close(tensor_to_bits(got), st.decode(w.q_dec[t], w.scale), f"static scratch, call {t}")
    s.close()


def test_static_scratch_on_a_prefix_aware_plan_twice():
    # two worker groups (G = 8, twenty workers): the shared-prefix scan's partials land in the fixed array too
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor, tensor_to_bits

    w = wl.prefix_aware(20, 128, 16, 2, 128, steps=2, seed=47).materialise()
    o = w.own
    dev = lambda a: bits_to_tensor(a, "cuda:0")
    shape = (w.num_pages, o.num_kv_heads, o.page_size, o.head_dim)
    pools = (torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda:0"),
             torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda:0"))
    hist = CompactionSession([w.hist_tokens], 0, o.num_q_heads, o.num_kv_heads, o.head_dim, w.shared_pages,
                             w.num_pages, scale=o.scale, pools=pools)
    hist.append_prefill(dev(w.k_hist), dev(w.v_hist))
    s = CompactionSession(o.block_lens, o.decode_steps, o.num_q_heads, o.num_kv_heads, o.head_dim, o.free_pages,
                          w.num_pages, scale=o.scale, prefix_lens=w.prefix_lens, shared_pages=w.shared_pages, pools=pools)
    assert s.param(B.PARAM_DECODE_WORKSPACE_BYTES) <= B.STATIC_SCRATCH_BYTES
    q0 = dev(o.q_dec[0])
    # no own token cached yet: nothing could merge the shared scan's partials, the call says so
    assert B.cpa_decode_static(s.plan, q0, s.k_pool, s.v_pool, torch.empty_like(q0)) == B.CPA_ESTATE
    assert B.cpa_decode(s.plan, q0, s.k_pool, s.v_pool, torch.empty_like(q0), s.workspace) == B.CPA_ESTATE
    s.append_prefill(dev(o.k), dev(o.v))
    cu = np.concatenate([[0], np.cumsum(o.block_lens.astype(np.int64))])
    st = oa.PrefixDecodeState(o.k, o.v, cu, w.k_hist, w.v_hist, w.prefix_lens, o.decode_steps)
    stream = int(torch.cuda.current_stream().cuda_stream)
    for t in range(2):
        s.append(dev(o.k_dec[t]), dev(o.v_dec[t]))
        st.append(o.k_dec[t], o.v_dec[t])
        q = dev(o.q_dec[t])
        want = s.decode(q)
        got = torch.full_like(want, 9.0)
        assert B.cpa_decode_static(s.plan, q, s.k_pool, s.v_pool, got, stream) == B.CPA_OK
        assert s.status() == 0
        assert np.array_equal(tensor_to_bits(got), tensor_to_bits(want)), f"call {t}: differs from cpa_decode"
        assert_attention_close(tensor_to_bits(got), st.decode(o.q_dec[t], o.scale), f"static scratch, prefix plan, call {t}")
    s.close()
    hist.close()


def test_static_scratch_rejects_plans_that_need_more_than_it_holds():
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession

    # 64 blocks x 32 heads with one page per split: far more partial rows than 16 MiB holds
    w = wl.custom([2048] * 64, 32, 8, 128, steps=0, seed=42)
    free = np.arange(w.num_pages, dtype=np.int32)
    s = CompactionSession(w.block_lens, 0, 32, 8, 128, free, w.num_pages, pages_per_split=1)
    assert s.param(B.PARAM_DECODE_WORKSPACE_BYTES) > B.STATIC_SCRATCH_BYTES
    q = torch.zeros((64, 32, 128), dtype=torch.bfloat16, device="cuda:0")
    o = torch.zeros_like(q)
    assert B.cpa_decode_static(s.plan, q, s.k_pool, s.v_pool, o) == B.CPA_ENOSPC
    s.close()
