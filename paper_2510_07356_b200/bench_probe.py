"""ctypes binding of libconcur_bench.so, the benchmark's helper library: a read-only stream over a
device buffer (the plain-stream yardstick the attention kernels are held against).  Not part of the
attention library; bench.py and the probe's own test load it."""
from __future__ import annotations

import ctypes
from pathlib import Path

_LIB_PATH = Path(__file__).resolve().parent / "libconcur_bench.so"
if not _LIB_PATH.exists():
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2510_07356_b200.build`")
lib = ctypes.CDLL(str(_LIB_PATH))
lib.concur_bench_read_probe.restype = ctypes.c_int
lib.concur_bench_read_probe.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_int32,
                                        ctypes.c_void_p]
ERR_INVALID_ARG = -1


def read_probe(buf, nbytes, checksum, ctas=0, stream=0, check=True) -> int:
    """Reads `nbytes` bytes of the device tensor `buf` once; xor of its 32-bit words -> checksum[0]."""
    addr = lambda x: 0 if x is None else (x if isinstance(x, int) else x.data_ptr())
    rc = lib.concur_bench_read_probe(addr(buf), int(nbytes), addr(checksum), int(ctas), stream or None)
    if check and rc != 0:
        raise RuntimeError(f"concur_bench_read_probe failed ({rc})")
    return rc
