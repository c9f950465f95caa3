"""ctypes front end of the float64 CPU oracle (TEST INFRASTRUCTURE).

Only tests, the smoke check and the bench's CPU-baseline leg import this
package.  It marshals numpy arrays into ``puzzle_oracle.c`` and does no
arithmetic of its own.  bf16 tensors travel as uint16 bit patterns.

The shared object is compiled from the C file next to this module with
``gcc`` the first time it is needed (or when the source is newer).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "puzzle_oracle.c")
_LIB = os.path.join(_HERE, "libpuzzle_oracle.so")
_lock = threading.Lock()
_lib = None

KV_FP8_E4M3 = 0
KV_BF16 = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; returns the path of the shared object."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.oracle_e4m3_decode.restype = ctypes.c_double
            lib.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
            lib.oracle_e4m3_encode.restype = ctypes.c_uint8
            lib.oracle_e4m3_encode.argtypes = [ctypes.c_float]
            _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _arr(a, dtype):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def host_cores() -> int:
    """Cores this process may run on (the thread count the oracle is given)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def e4m3_decode(code: int) -> float:
    return float(_load().oracle_e4m3_decode(int(code) & 0xFF))


def e4m3_encode(y: float) -> int:
    return int(_load().oracle_e4m3_encode(ctypes.c_float(y)))


def e4m3_encode_array(y) -> np.ndarray:
    y = np.ascontiguousarray(y, dtype=np.float32)
    out = np.empty(y.shape, dtype=np.uint8)
    _load().oracle_e4m3_encode_array(_ptr(y), ctypes.c_int64(y.size), _ptr(out))
    return out


def calibrate_scales(x, pow2: bool = False) -> np.ndarray:
    """x: float32 [n_tokens][Hkv][D] -> float32 [Hkv] scales (amax/448)."""
    x = _arr(x, np.float32)
    n, hkv, d = x.shape
    out = np.empty(hkv, dtype=np.float32)
    _load().oracle_calibrate_scales(
        _ptr(x), ctypes.c_int64(n), ctypes.c_int(hkv), ctypes.c_int(d), ctypes.c_int(int(pow2)), _ptr(out)
    )
    return out


def kv_append(k_cache, v_cache, kv_dtype, block_size, block_table, max_blocks_per_seq, seq_lens,
              k_scale, v_scale, k_new, v_new) -> None:
    """In-place append into numpy caches [num_blocks][Hkv][block_size][D]."""
    cdt = np.uint8 if kv_dtype == KV_FP8_E4M3 else np.uint16
    assert k_cache.dtype == cdt and v_cache.dtype == cdt
    assert k_cache.flags["C_CONTIGUOUS"] and v_cache.flags["C_CONTIGUOUS"]
    _, hkv, bs, d = k_cache.shape
    assert bs == block_size
    block_table = _arr(block_table, np.int32)
    seq_lens = _arr(seq_lens, np.int32)
    k_scale = _arr(k_scale, np.float32)
    v_scale = _arr(v_scale, np.float32)
    k_new = _arr(k_new, np.uint16)
    v_new = _arr(v_new, np.uint16)
    batch = seq_lens.shape[0]
    assert k_new.shape == (batch, hkv, d) and v_new.shape == (batch, hkv, d)
    _load().oracle_kv_append(
        _ptr(k_cache), _ptr(v_cache), ctypes.c_int(kv_dtype), ctypes.c_int(hkv), ctypes.c_int(d),
        ctypes.c_int(block_size), _ptr(block_table), ctypes.c_int(max_blocks_per_seq), _ptr(seq_lens),
        _ptr(k_scale), _ptr(v_scale), _ptr(k_new), _ptr(v_new), ctypes.c_int(batch),
    )


def _items(items, batch, hq):
    if items is None:
        items = [(b, g) for b in range(batch) for g in range(hq)]
    items = np.ascontiguousarray(np.asarray(items, dtype=np.int32).reshape(-1, 2))
    return items


def decode_attn(k_cache, v_cache, kv_dtype, block_table, max_blocks_per_seq, seq_lens, k_scale,
                v_scale, q, sinks, window, sm_scale, items=None, threads=None):
    """Returns (out float64 [n_items][D], lse float64 [n_items]).

    ``items`` lists (sequence, query head) pairs; None means all, ordered
    [batch][Hq], so the result reshapes to [batch][Hq][D].
    """
    _, hkv, bs, d = k_cache.shape
    q = _arr(q, np.uint16)
    batch, hq, dq = q.shape
    assert dq == d
    block_table = _arr(block_table, np.int32)
    seq_lens = _arr(seq_lens, np.int32)
    k_scale = _arr(k_scale, np.float32)
    v_scale = _arr(v_scale, np.float32)
    sinks = _arr(sinks, np.float32)
    items = _items(items, batch, hq)
    n = items.shape[0]
    out = np.zeros((n, d), dtype=np.float64)
    lse = np.zeros(n, dtype=np.float64)
    _load().oracle_decode_attn(
        _ptr(k_cache), _ptr(v_cache), ctypes.c_int(kv_dtype), ctypes.c_int(hq), ctypes.c_int(hkv),
        ctypes.c_int(d), ctypes.c_int(bs), _ptr(block_table), ctypes.c_int(max_blocks_per_seq),
        _ptr(seq_lens), _ptr(k_scale), _ptr(v_scale), _ptr(q), _ptr(sinks), ctypes.c_int(int(window)),
        ctypes.c_double(sm_scale), _ptr(items), ctypes.c_int64(n), _ptr(out), _ptr(lse),
        ctypes.c_int(threads or host_cores()),
    )
    return out, lse


def partial_attn(k_cache, v_cache, kv_dtype, block_table, max_blocks_per_seq, seq_lens, k_scale,
                 v_scale, q, sm_scale, t0, t1, items=None, threads=None):
    """Attention over keys [t0, t1) only, without sink: (out, lse) of one split."""
    _, hkv, bs, d = k_cache.shape
    q = _arr(q, np.uint16)
    batch, hq, _ = q.shape
    block_table = _arr(block_table, np.int32)
    seq_lens = _arr(seq_lens, np.int32)
    k_scale = _arr(k_scale, np.float32)
    v_scale = _arr(v_scale, np.float32)
    items = _items(items, batch, hq)
    n = items.shape[0]
    out = np.zeros((n, d), dtype=np.float64)
    lse = np.zeros(n, dtype=np.float64)
    _load().oracle_partial_attn(
        _ptr(k_cache), _ptr(v_cache), ctypes.c_int(kv_dtype), ctypes.c_int(hq), ctypes.c_int(hkv),
        ctypes.c_int(d), ctypes.c_int(bs), _ptr(block_table), ctypes.c_int(max_blocks_per_seq),
        _ptr(seq_lens), _ptr(k_scale), _ptr(v_scale), _ptr(q), ctypes.c_double(sm_scale),
        ctypes.c_int64(int(t0)), ctypes.c_int64(int(t1)), _ptr(items), ctypes.c_int64(n), _ptr(out),
        _ptr(lse), ctypes.c_int(threads or host_cores()),
    )
    return out, lse


def attn_merge(part_o, part_lse, num_parts=None, sink=None):
    """part_o [rows][S][D], part_lse [rows][S] -> (out [rows][D], lse [rows])."""
    part_o = _arr(part_o, np.float64)
    part_lse = _arr(part_lse, np.float64)
    rows, s, d = part_o.shape
    assert part_lse.shape == (rows, s)
    num_parts = _arr(num_parts, np.int32)
    sink = _arr(sink, np.float64)
    out = np.zeros((rows, d), dtype=np.float64)
    lse = np.zeros(rows, dtype=np.float64)
    _load().oracle_attn_merge(
        _ptr(part_o), _ptr(part_lse), _ptr(num_parts), _ptr(sink), ctypes.c_int64(rows),
        ctypes.c_int(s), ctypes.c_int(d), _ptr(out), _ptr(lse),
    )
    return out, lse
