"""ctypes binding of libconcur_attn.so: the same names as include/concur_attn.h.

Argument marshalling only -- every step of the decode-attention path (plan, partial,
combine) runs in the library's CUDA kernels.  There is no fallback: if the shared
library is missing or was not built, importing this module raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import os

# CONCUR_ATTN_LIBRARY names another build of the same library to load instead -- the checked build
# (libconcur_attn_bounds.so), whose kernels verify every index they compute; there is no other use.
_LIB_PATH = Path(os.environ.get("CONCUR_ATTN_LIBRARY") or Path(__file__).resolve().parent / "libconcur_attn.so")

CONCUR_OK = 0
CONCUR_ERR_INVALID_ARG = -1
CONCUR_ERR_UNSUPPORTED = -2
CONCUR_ERR_TOO_LARGE = -3
CONCUR_ERR_CUDA = -4
CONCUR_ERR_OOM = -5

CONCUR_FLAG_BAD_PAGE_ID = 1
CONCUR_FLAG_BAD_SEQ_LEN = 2
CONCUR_FLAG_WAIT_LIMIT = 4
CONCUR_FLAG_BAD_GROUP = 8
CONCUR_FLAG_BOUNDS = 16

CONCUR_KV_HEAD_MAJOR = 0
CONCUR_KV_TOKEN_MAJOR = 1

CONCUR_OPT_KERNEL = 1
CONCUR_OPT_NUM_RANGES = 2
CONCUR_OPT_GRID_CTAS = 3
CONCUR_OPT_RANGES_PER_CTA = 4
CONCUR_OPT_MIN_RANGE_TILES = 5
CONCUR_OPT_EVENT_BEFORE_PARTIAL = 6
CONCUR_OPT_EVENT_AFTER_PARTIAL = 7
CONCUR_OPT_FUSE_COMBINE = 8
CONCUR_OPT_CLAIM_AHEAD = 9
CONCUR_OPT_PREFIX_KERNEL = 10
CONCUR_OPT_SMALL_PAGE_COPY = 11
CONCUR_OPT_WAIT_LIMIT_NS = 12
CONCUR_OPT_OVERLAP_CALLS = 13
CONCUR_OPT_PREFILL_KERNEL = 14

EXPORTS = (
    "concur_attn_workspace_bytes", "concur_attn_create", "concur_decode_attn",
    "concur_decode_attn_host", "concur_attn_status", "concur_attn_set_option",
    "concur_attn_last_plan", "concur_attn_destroy", "concur_attn_strerror",
    "concur_decode_attn_static", "concur_kv_append", "concur_decode_attn_cascade", "concur_prefill_attn",
    "concur_curate", "concur_attn_plan", "concur_decode_attn_planned",
    "concur_kv_append_layer", "concur_decode_attn_append", "concur_lse_merge",
)
CONCUR_STATIC_MAX_BATCH = 1024
CONCUR_STATIC_MAX_RANGES = 512


class concur_attn_config_t(ctypes.Structure):
    _fields_ = [
        ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("max_batch", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
        ("device", ctypes.c_int32), ("kv_layout", ctypes.c_int32),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
    ]


class concur_curate_params_t(ctypes.Structure):
    _fields_ = [
        ("num_tasks", ctypes.c_int32), ("gens", ctypes.c_int32), ("rule_b_speedup", ctypes.c_float),
        ("fast_p", ctypes.c_float), ("top_k", ctypes.c_int32), ("easy_below", ctypes.c_int32),
        ("hard_above", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]


CONCUR_SEL_RANDOM, CONCUR_SEL_MAX_LENGTH, CONCUR_SEL_MIN_LENGTH, CONCUR_SEL_SPEEDUP = 0, 1, 2, 3
(CONCUR_STAT_CORRECT, CONCUR_STAT_TASKS_CORRECT, CONCUR_STAT_RULE_A, CONCUR_STAT_RULE_B, CONCUR_STAT_LENGTH_SUM,
 CONCUR_STAT_ARL, CONCUR_STAT_FAST_FIRST_COUNT, CONCUR_STAT_FAST_BEST_COUNT, CONCUR_STAT_EXEC_FIRST_COUNT,
 CONCUR_STAT_N, CONCUR_STAT_SX, CONCUR_STAT_SY, CONCUR_STAT_SXX, CONCUR_STAT_SYY, CONCUR_STAT_SXY,
 CONCUR_STAT_PEARSON_R, CONCUR_STAT_FAST_FIRST, CONCUR_STAT_FAST_BEST) = range(18)
CONCUR_CURATE_NUM_STATS = 24


def _load() -> ctypes.CDLL:
    if not _LIB_PATH.exists():
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2510_07356_b200.build` "
            "(nvcc, sm_100a). There is no CPU or PyTorch fallback.")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i32, i32p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)
    cfgp = ctypes.POINTER(concur_attn_config_t)
    lib.concur_attn_workspace_bytes.restype = ctypes.c_size_t
    lib.concur_attn_workspace_bytes.argtypes = [cfgp]
    lib.concur_attn_create.restype = ctypes.c_int
    lib.concur_attn_create.argtypes = [cfgp, ctypes.POINTER(vp)]
    decode_args = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, i32, i32, i32, vp]
    lib.concur_decode_attn.restype = ctypes.c_int
    lib.concur_decode_attn.argtypes = decode_args
    lib.concur_decode_attn_planned.restype = ctypes.c_int
    lib.concur_decode_attn_planned.argtypes = decode_args
    lib.concur_attn_plan.restype = ctypes.c_int
    lib.concur_attn_plan.argtypes = [vp, vp, i32, i32, vp]
    lib.concur_decode_attn_host.restype = ctypes.c_int
    lib.concur_decode_attn_host.argtypes = decode_args
    lib.concur_decode_attn_static.restype = ctypes.c_int
    lib.concur_decode_attn_static.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, i32, i32, i32, i32, vp]
    lib.concur_decode_attn_cascade.restype = ctypes.c_int
    lib.concur_decode_attn_cascade.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp,
                                               i32, i32, i32, i32, vp]
    lib.concur_curate.restype = ctypes.c_int
    lib.concur_curate.argtypes = [ctypes.POINTER(concur_curate_params_t)] + [vp] * 14
    lib.concur_prefill_attn.restype = ctypes.c_int
    lib.concur_prefill_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, i32, i32, i32, i32, vp]
    lib.concur_kv_append.restype = ctypes.c_int
    lib.concur_kv_append.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp]
    lib.concur_decode_attn_append.restype = ctypes.c_int
    lib.concur_decode_attn_append.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, i32, i32, i32, vp]
    lib.concur_lse_merge.restype = ctypes.c_int
    lib.concur_lse_merge.argtypes = [vp, vp, i32, ctypes.c_int64, vp, vp, vp]
    lib.concur_kv_append_layer.restype = ctypes.c_int
    lib.concur_kv_append_layer.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.concur_attn_status.restype = ctypes.c_int
    lib.concur_attn_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.concur_attn_set_option.restype = ctypes.c_int
    lib.concur_attn_set_option.argtypes = [vp, i32, ctypes.c_int64]
    lib.concur_attn_last_plan.restype = ctypes.c_int
    lib.concur_attn_last_plan.argtypes = [vp, vp, i32p, i32p, i32p, i32]
    lib.concur_attn_destroy.restype = ctypes.c_int
    lib.concur_attn_destroy.argtypes = [vp]
    lib.concur_attn_strerror.restype = ctypes.c_char_p
    lib.concur_attn_strerror.argtypes = [ctypes.c_int]
    return lib


lib = _load()


class ConcurError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {concur_attn_strerror(code)} ({code})")


def concur_attn_strerror(code: int) -> str:
    return lib.concur_attn_strerror(int(code)).decode()


def make_config(page_size: int, max_batch: int, max_pages_per_seq: int, device: int = 0,
                num_q_heads: int = 64, num_kv_heads: int = 8, head_dim: int = 128,
                workspace: int = 0, workspace_bytes: int = 0, kv_layout: int = 0) -> concur_attn_config_t:
    return concur_attn_config_t(num_q_heads, num_kv_heads, head_dim, page_size, max_batch,
                                max_pages_per_seq, device, kv_layout, workspace or None, workspace_bytes)


def concur_attn_workspace_bytes(cfg: concur_attn_config_t) -> int:
    return int(lib.concur_attn_workspace_bytes(ctypes.byref(cfg)))


def concur_attn_create(cfg: concur_attn_config_t) -> int:
    """Returns the handle as an integer address; raises ConcurError on failure."""
    h = ctypes.c_void_p()
    rc = lib.concur_attn_create(ctypes.byref(cfg), ctypes.byref(h))
    if rc != CONCUR_OK:
        raise ConcurError(rc, "concur_attn_create")
    return h.value


def _addr(x) -> int:
    """Device or host address of a torch tensor / numpy array / int."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return x.ctypes.data


def _decode(fn, name, handle, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse,
            batch, num_pages, block_table_stride, stream, check):
    rc = fn(handle, _addr(q), _addr(k_pages), _addr(v_pages), _addr(block_table), _addr(seq_lens),
            ctypes.c_float(scale), _addr(out), _addr(lse), batch, num_pages, block_table_stride,
            stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, name)
    return rc


def concur_decode_attn(handle, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse,
                       batch, num_pages, block_table_stride, stream=0, check=True) -> int:
    """Device tensors (or raw device addresses); `stream` is a cudaStream_t as an int."""
    return _decode(lib.concur_decode_attn, "concur_decode_attn", handle, q, k_pages, v_pages,
                   block_table, seq_lens, scale, out, lse, batch, num_pages, block_table_stride,
                   stream, check)


def concur_attn_plan(handle, seq_lens, batch, block_table_stride, stream=0, check=True) -> int:
    """The split-KV plan of one token step, for the concur_decode_attn_planned calls of its layers."""
    rc = lib.concur_attn_plan(handle, _addr(seq_lens), batch, block_table_stride, stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_attn_plan")
    return rc


def concur_decode_attn_planned(handle, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse,
                               batch, num_pages, block_table_stride, stream=0, check=True) -> int:
    """concur_decode_attn as one launch, on the plan of the preceding concur_attn_plan call."""
    return _decode(lib.concur_decode_attn_planned, "concur_decode_attn_planned", handle, q, k_pages, v_pages,
                   block_table, seq_lens, scale, out, lse, batch, num_pages, block_table_stride,
                   stream, check)


def concur_decode_attn_host(handle, q, k_pages, v_pages, block_table, seq_lens, scale, out, lse,
                            batch, num_pages, block_table_stride, stream=0, check=True) -> int:
    """Host tensors (pinned for asynchronous copies); synchronises before returning."""
    return _decode(lib.concur_decode_attn_host, "concur_decode_attn_host", handle, q, k_pages,
                   v_pages, block_table, seq_lens, scale, out, lse, batch, num_pages,
                   block_table_stride, stream, check)


def concur_decode_attn_static(q, k_pages, v_pages, block_table, seq_lens, scale, out, lse,
                              batch, num_pages, block_table_stride, page_size, stream=0, check=True) -> int:
    """The handle-free variant for callers that must not allocate device memory: its
    workspace is a fixed array inside the library.  Device tensors; current device; calls
    must not overlap on the GPU (they share that array)."""
    rc = lib.concur_decode_attn_static(_addr(q), _addr(k_pages), _addr(v_pages), _addr(block_table),
                                       _addr(seq_lens), ctypes.c_float(scale), _addr(out), _addr(lse),
                                       batch, num_pages, block_table_stride, page_size, stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_decode_attn_static")
    return rc


def concur_decode_attn_cascade(handle, q, k_pages, v_pages, block_table, seq_lens, group_start, prefix_lens,
                               scale, out, lse, batch, num_groups, num_pages, block_table_stride,
                               stream=0, check=True) -> int:
    """Decode attention for groups of sequences that share a cached prefix (device tensors)."""
    rc = lib.concur_decode_attn_cascade(handle, _addr(q), _addr(k_pages), _addr(v_pages), _addr(block_table),
                                        _addr(seq_lens), _addr(group_start), _addr(prefix_lens),
                                        ctypes.c_float(scale), _addr(out), _addr(lse), batch, num_groups,
                                        num_pages, block_table_stride, stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_decode_attn_cascade")
    return rc


def concur_prefill_attn(handle, q, k_pages, v_pages, block_table, seq_lens, q_start, scale, out, lse, batch,
                        total_q, num_pages, block_table_stride, stream=0, check=True) -> int:
    """Causal attention of each sequence's last q_len cached tokens (device tensors)."""
    rc = lib.concur_prefill_attn(handle, _addr(q), _addr(k_pages), _addr(v_pages), _addr(block_table),
                                 _addr(seq_lens), _addr(q_start), ctypes.c_float(scale), _addr(out), _addr(lse),
                                 batch, total_q, num_pages, block_table_stride, stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_prefill_attn")
    return rc


def concur_curate(params: concur_curate_params_t, correct, t_torch, t_kernel, length, sample_key, task_key,
                  speedup, rule_a, rule_b, pick, keep, difficulty, stats, stream=0, check=True) -> int:
    """Curation arithmetic over [N][M] generation records (device tensors; see include/concur_curate.h)."""
    rc = lib.concur_curate(ctypes.byref(params), _addr(correct), _addr(t_torch), _addr(t_kernel), _addr(length),
                           _addr(sample_key), _addr(task_key), _addr(speedup), _addr(rule_a), _addr(rule_b),
                           _addr(pick), _addr(keep), _addr(difficulty), _addr(stats), stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_curate")
    return rc


def concur_kv_append(handle, k_new, v_new, k_pages, v_pages, block_table, seq_lens, batch, num_pages,
                     block_table_stride, stream=0, check=True) -> int:
    """Stores each sequence's new K/V rows at position seq_lens[b] and advances seq_lens (device tensors)."""
    rc = lib.concur_kv_append(handle, _addr(k_new), _addr(v_new), _addr(k_pages), _addr(v_pages),
                              _addr(block_table), _addr(seq_lens), batch, num_pages, block_table_stride,
                              stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_kv_append")
    return rc


def concur_kv_append_layer(handle, k_new, v_new, k_pages, v_pages, block_table, seq_lens, batch, num_pages,
                           block_table_stride, advance, stream=0, check=True) -> int:
    """concur_kv_append for one layer of several: advance=1 for the step's first append, 0 for the others
    (they write the slot the first one opened and leave seq_lens alone)."""
    rc = lib.concur_kv_append_layer(handle, _addr(k_new), _addr(v_new), _addr(k_pages), _addr(v_pages),
                                    _addr(block_table), _addr(seq_lens), batch, num_pages, block_table_stride,
                                    int(advance), stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_kv_append_layer")
    return rc


def concur_decode_attn_append(handle, q, k_new, v_new, k_pages, v_pages, block_table, seq_lens, scale, out, lse,
                              batch, num_pages, block_table_stride, stream=0, check=True) -> int:
    """Append (without advancing seq_lens) and attend in one launch: the newest token's rows come from
    k_new / v_new and are stored into the pools by the attention kernel."""
    rc = lib.concur_decode_attn_append(handle, _addr(q), _addr(k_new), _addr(v_new), _addr(k_pages), _addr(v_pages),
                                       _addr(block_table), _addr(seq_lens), ctypes.c_float(scale), _addr(out),
                                       _addr(lse), batch, num_pages, block_table_stride, stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_decode_attn_append")
    return rc


def concur_lse_merge(outs, lses, parts, rows, out, lse, stream=0, check=True) -> int:
    """Merges `parts` attention results of the same query rows over different key ranges (device tensors:
    outs bf16 [parts][rows][D], lses fp32 [parts][rows]) into out [rows][D], lse [rows]."""
    rc = lib.concur_lse_merge(_addr(outs), _addr(lses), int(parts), int(rows), _addr(out), _addr(lse), stream or None)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_lse_merge")
    return rc


def concur_attn_status(handle, stream=0) -> int:
    flags = ctypes.c_uint32(0)
    rc = lib.concur_attn_status(handle, stream or None, ctypes.byref(flags))
    if rc != CONCUR_OK:
        raise ConcurError(rc, "concur_attn_status")
    return flags.value


def concur_attn_set_option(handle, key: int, value: int, check=True) -> int:
    rc = lib.concur_attn_set_option(handle, key, value)
    if check and rc != CONCUR_OK:
        raise ConcurError(rc, "concur_attn_set_option")
    return rc


def concur_attn_last_plan(handle, stream=0, cap: int = 8192):
    """Returns (num_ranges, total_tiles, range_start list) of the most recent call."""
    n, w = ctypes.c_int32(0), ctypes.c_int32(0)
    buf = (ctypes.c_int32 * cap)()
    rc = lib.concur_attn_last_plan(handle, stream or None, ctypes.byref(n), ctypes.byref(w), buf, cap)
    if rc != CONCUR_OK:
        raise ConcurError(rc, "concur_attn_last_plan")
    return n.value, w.value, list(buf[: min(cap, n.value + 1)])


def concur_attn_destroy(handle) -> int:
    return lib.concur_attn_destroy(handle)
