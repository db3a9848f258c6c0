"""Binding of the benchmark's row-gather probe (``libtiga_bench_probe.so``, built by
``paper_2609_24802_b200.build``).  It is a measuring device of ``bench.py`` -- the L2 -> SM gather
ceiling and the time of a workload's gathers alone -- and not part of the library's C ABI."""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtiga_bench_probe.so")
_lib = None
launches = 0


def load():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_24802_b200.build`")
        _lib = ctypes.CDLL(LIB_PATH)
        vp = ctypes.c_void_p
        _lib.tiga_bench_probe_row_gather.restype = ctypes.c_int
        _lib.tiga_bench_probe_row_gather.argtypes = [vp, ctypes.c_int64, ctypes.c_int32, vp, ctypes.c_int64, vp, vp]
    return _lib


def row_gather(table, idx, sink, stream=None) -> None:
    """Gathers table[idx[k], :] for every k (rows of 16..512 bytes) and folds them into sink[0]."""
    global launches
    s = torch.cuda.current_stream() if stream is None else stream
    st = load().tiga_bench_probe_row_gather(table.data_ptr(), table.shape[0], table.shape[1] * table.element_size(),
                                            idx.data_ptr(), idx.numel(), sink.data_ptr(), s.cuda_stream)
    if st != 0:
        raise ValueError(f"tiga_bench_probe_row_gather: status {st}")
    launches += 1
