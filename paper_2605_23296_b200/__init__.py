"""libcompact_attn for B200: attention hot path of parallel context compaction.

``binding``    ctypes layer over the C-ABI library (loaded on first use)
``workloads``  seeded synthetic inputs (no attention arithmetic)
``build``      in-tree nvcc build of the library
"""


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
