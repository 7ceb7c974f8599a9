"""The give-up path of the kernels' bounded waits, executed once in the one harmless form there is: a
test-only kernel (its own shared library, not part of libcompact_attn) waits with the library's wait
routine, with a limit of a thousand tries, on an mbarrier that nothing arrives at.  The wait must run
out, the kernel must return, and the plan's status word must read back as CPA_ETIMEOUT.  Nothing here
faults, traps or hangs the device."""
import ctypes
import os

import numpy as np
import pytest

from paper_2605_23296_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_sets_the_status_word_and_returns():
    import torch
    from paper_2605_23296_b200 import binding as B
    from paper_2605_23296_b200 import build
    from paper_2605_23296_b200.session import CompactionSession

    probe = ctypes.CDLL(build.PROBE_LIB)
    probe.cpa_test_wait_probe.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p]
    probe.cpa_test_wait_probe.restype = ctypes.c_int

    w = wl.tiny(3).materialise()
    s = CompactionSession(w.block_lens, w.decode_steps, w.num_q_heads, w.num_kv_heads, w.head_dim, w.free_pages,
                          w.num_pages, scale=w.scale)
    assert s.status() == B.CPA_OK
    trace = torch.zeros(4, dtype=torch.int32, device="cuda:0")
    stream = int(torch.cuda.current_stream().cuda_stream)
    # the status word is the first int32 of the plan's index buffer
    assert probe.cpa_test_wait_probe(s.index_buf.data_ptr(), trace.data_ptr(), 1000, stream) == 0
    torch.cuda.synchronize()
    # (wait completed, dead flag, second wait completed, kernel reached its end)
    assert trace.cpu().tolist() == [0, 1, 0, 1]
    assert s.status() == B.CPA_ETIMEOUT
    assert "wait" in B.cpa_strerror(s.status())
    # the first code recorded stays: a later "no room" does not overwrite a timeout ...
    word = s.index_buf[:4].view(torch.int32)
    assert int(word.item()) == 1
    # ... and a plan whose word holds the append's code reads back as CPA_ENOSPC
    word.fill_(2)
    assert s.status() == B.CPA_ENOSPC
    # uploading the plan again clears the word; the plan works again
    s._check(B.cpa_plan_upload(s.plan, s.index_buf, s.index_buf.numel(), stream), "cpa_plan_upload")
    assert s.status() == B.CPA_OK
    s.close()
