"""cpa_decode_static: the decode entry point for callers that cannot provide scratch memory
(for instance a plugin limited to the buffers its host framework gave it, or a service whose
device memory was budgeted in full at start-up).  Its split partials live in a fixed array
inside the library, so its results must equal cpa_decode's, call after call, although the
array keeps old contents.

Collected last on purpose: a run that stops at the first failure has then already run
every other test."""
import numpy as np
import pytest

from _util import MAX_ABS, bits_to_f64
from paper_2605_23296_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_twice():
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200.session import CompactionSession, bits_to_tensor, tensor_to_bits

    w = wl.custom([700, 33, 257, 1200], 8, 2, 128, steps=3, seed=41).materialise()
    s = CompactionSession(w.block_lens, w.decode_steps, w.num_q_heads, w.num_kv_heads, w.head_dim,
                          w.free_pages, w.num_pages, scale=w.scale, poison_pools=True)
    assert s.param(B.PARAM_DECODE_WORKSPACE_BYTES) <= B.STATIC_SCRATCH_BYTES
    dev = lambda a: bits_to_tensor(a, "cuda:0")
    s.append_prefill(dev(w.k), dev(w.v))
    stream = int(torch.cuda.current_stream().cuda_stream)
    for t in range(2):          # two calls in a row: the second one finds the first one's partials
        s.append(dev(w.k_dec[t]), dev(w.v_dec[t]))
        q = dev(w.q_dec[t])
        want = s.decode(q)
        got = torch.full_like(want, 9.0)
        rc = B.cpa_decode_static(s.plan, q, s.k_pool, s.v_pool, got, stream)
        assert rc == B.CPA_OK, B.cpa_strerror(rc)
        assert s.status() == 0
        a, b = bits_to_f64(tensor_to_bits(got)), bits_to_f64(tensor_to_bits(want))
        assert np.isfinite(a).all()
        assert np.abs(a - b).max() <= MAX_ABS, f"call {t}: {np.abs(a - b).max()}"
    s.close()


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
