"""CPU oracle for the compaction attention path.  TEST INFRASTRUCTURE ONLY.

Nothing here is part of the product: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  It shares no code with the CUDA
path and never imports it.

Modules
-------
plan       index construction (cu_seqlens, page table, slots, work lists)
attention  fp64 attention by the plain definition (C core, loaded via ctypes),
           contiguous-KV decode state, expected pool contents, split combine
"""
