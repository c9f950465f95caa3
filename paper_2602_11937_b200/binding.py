"""ctypes binding of the C ABI: same entry-point names, argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "lib", "libpuzzle_attn.so")
_lib = None

KV_FP8_E4M3 = 0
KV_BF16 = 1
DEV_BAD_BLOCK = 1
DEV_SEQ_TOO_LONG = 2
DEV_WAIT_EXPIRED = 4
STATIC_SCRATCH_BYTES = 8 << 20
SCHED_AUTO, SCHED_CTA, SCHED_WARP = 0, -1, -2      # num_splits values that select the balanced schedule

EXPORTS = (
    "puzzle_kv_amax_update",
    "puzzle_kv_scales_from_amax",
    "puzzle_kv_append",
    "puzzle_kv_append_tokens",
    "puzzle_decode_attn_workspace_bytes",
    "puzzle_decode_attn_workspace_init",
    "puzzle_decode_attn",
    "puzzle_decode_attn_tcgen05",
    "puzzle_decode_attn_static",
    "puzzle_decode_attn_partial",
    "puzzle_decode_step_host",
    "puzzle_decode_step_host_staging_bytes",
    "puzzle_decode_attn_tokens",
    "puzzle_decode_attn_tokens_workspace_bytes",
    "puzzle_decode_attn_tokens_workspace_init",
    "puzzle_attn_merge",
    "puzzle_attn_merge_strided",
    "puzzle_hbm_read_probe",
    "puzzle_status_string",
    "puzzle_launch_count",
    "puzzle_decode_attn_kernel_name",
)


class PuzzleError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: status %d (%s)" % (where, code, puzzle_status_string(code)))


class LayerDesc(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("block_size", ctypes.c_int32), ("window", ctypes.c_int32), ("kv_dtype", ctypes.c_int32),
                ("sm_scale", ctypes.c_float)]


class KVView(ctypes.Structure):
    _fields_ = [("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p), ("num_blocks", ctypes.c_int64),
                ("block_table", ctypes.c_void_p), ("max_blocks_per_seq", ctypes.c_int32),
                ("seq_lens", ctypes.c_void_p), ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p)]


def library_path() -> str:
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                "CUDA library %s is missing: build it with `python -m paper_2602_11937_b200.build` "
                "(there is no CPU fallback)" % _LIB_PATH)
        lib = ctypes.CDLL(_LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        lib.puzzle_kv_append.restype = ctypes.c_int
        lib.puzzle_kv_append.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(KVView), vp, vp, i32, vp, vp]
        lib.puzzle_kv_amax_update.restype = ctypes.c_int
        lib.puzzle_kv_amax_update.argtypes = [vp, ctypes.c_int64, i32, i32, vp, vp]
        lib.puzzle_kv_scales_from_amax.restype = ctypes.c_int
        lib.puzzle_kv_scales_from_amax.argtypes = [vp, i32, i32, vp, vp]
        lib.puzzle_kv_append_tokens.restype = ctypes.c_int
        lib.puzzle_kv_append_tokens.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(KVView), vp, vp, vp, i32, i32,
                                                vp, vp]
        lib.puzzle_decode_attn_workspace_bytes.restype = sz
        lib.puzzle_decode_attn_workspace_bytes.argtypes = [ctypes.POINTER(LayerDesc), i32, i32]
        lib.puzzle_decode_attn_workspace_init.restype = ctypes.c_int
        lib.puzzle_decode_attn_workspace_init.argtypes = [ctypes.POINTER(LayerDesc), i32, vp, sz, vp]
        lib.puzzle_decode_attn.restype = ctypes.c_int
        lib.puzzle_decode_attn.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(KVView), vp, vp, vp, vp, i32, i32,
                                           vp, sz, vp, vp]
        lib.puzzle_decode_attn_tcgen05.restype = ctypes.c_int
        lib.puzzle_decode_attn_tcgen05.argtypes = lib.puzzle_decode_attn.argtypes
        lib.puzzle_decode_attn_partial.restype = ctypes.c_int
        lib.puzzle_decode_attn_partial.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(KVView), vp, vp, vp, i32, i32,
                                                   vp, sz, vp, vp]
        lib.puzzle_attn_merge_strided.restype = ctypes.c_int
        lib.puzzle_attn_merge_strided.argtypes = [vp, vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                                  vp, vp, vp, vp, i32, i32, i32, i32, vp]
        lib.puzzle_decode_attn_static.restype = ctypes.c_int
        lib.puzzle_decode_attn_static.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(KVView), vp, vp, vp, vp,
                                                  i32, i32, vp, vp]
        lib.puzzle_decode_step_host_staging_bytes.restype = sz
        lib.puzzle_decode_step_host_staging_bytes.argtypes = [ctypes.POINTER(LayerDesc), i32]
        lib.puzzle_decode_step_host.restype = ctypes.c_int
        lib.puzzle_decode_step_host.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(KVView), vp, vp, vp, vp, vp,
                                                i32, i32, vp, sz, vp, sz, vp, vp]
        lib.puzzle_decode_attn_tokens_workspace_bytes.restype = sz
        lib.puzzle_decode_attn_tokens_workspace_bytes.argtypes = [ctypes.POINTER(LayerDesc), i32, i32]
        lib.puzzle_decode_attn_tokens_workspace_init.restype = ctypes.c_int
        lib.puzzle_decode_attn_tokens_workspace_init.argtypes = [ctypes.POINTER(LayerDesc), i32, i32, vp, sz, vp]
        lib.puzzle_decode_attn_tokens.restype = ctypes.c_int
        lib.puzzle_decode_attn_tokens.argtypes = [ctypes.POINTER(LayerDesc), ctypes.POINTER(KVView), vp, vp, vp, vp, vp,
                                                  i32, i32, vp, sz, vp, vp]
        lib.puzzle_attn_merge.restype = ctypes.c_int
        lib.puzzle_attn_merge.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, vp]
        lib.puzzle_hbm_read_probe.restype = ctypes.c_int
        lib.puzzle_hbm_read_probe.argtypes = [vp, sz, vp, vp]
        lib.puzzle_status_string.restype = ctypes.c_char_p
        lib.puzzle_status_string.argtypes = [ctypes.c_int]
        lib.puzzle_launch_count.restype = ctypes.c_int64
        lib.puzzle_launch_count.argtypes = []
        lib.puzzle_decode_attn_kernel_name.restype = ctypes.c_char_p
        lib.puzzle_decode_attn_kernel_name.argtypes = [vp, vp, i32, i32]
        _lib = lib
    return _lib


def _p(t: Optional[torch.Tensor], dtype=None, name="tensor"):
    """Device pointer of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor" % name)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if dtype is not None and t.dtype != dtype:
        raise ValueError("%s must be %s, got %s" % (name, dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def layer_desc(window: int = 0, kv_dtype: int = KV_FP8_E4M3, num_q_heads: int = 64, num_kv_heads: int = 8,
               head_dim: int = 64, block_size: int = 16, sm_scale: Optional[float] = None) -> LayerDesc:
    return LayerDesc(num_q_heads, num_kv_heads, head_dim, block_size, int(window), int(kv_dtype),
                     float(sm_scale if sm_scale is not None else head_dim ** -0.5))


def kv_view(k_cache: torch.Tensor, v_cache: torch.Tensor, seq_lens: torch.Tensor,
            block_table: Optional[torch.Tensor] = None, max_blocks_per_seq: Optional[int] = None,
            k_scale: Optional[torch.Tensor] = None, v_scale: Optional[torch.Tensor] = None) -> KVView:
    """Describe one layer's cache ([num_blocks][Hkv][16][D], uint8 codes or bf16) for this batch.

    The view holds raw pointers: keep the tensors alive while it is in use."""
    if block_table is not None:
        max_blocks_per_seq = block_table.shape[1]
    if max_blocks_per_seq is None:
        raise ValueError("max_blocks_per_seq is required without a block table")
    v = KVView()
    v.k_cache = k_cache.data_ptr() if k_cache.is_cuda and k_cache.is_contiguous() else None
    v.v_cache = v_cache.data_ptr() if v_cache.is_cuda and v_cache.is_contiguous() else None
    v.num_blocks = k_cache.shape[0]
    v.block_table = _p(block_table, torch.int32, "block_table")
    v.max_blocks_per_seq = int(max_blocks_per_seq)
    v.seq_lens = _p(seq_lens, torch.int32, "seq_lens")
    v.k_scale = _p(k_scale, torch.float32, "k_scale")
    v.v_scale = _p(v_scale, torch.float32, "v_scale")
    return v


def puzzle_status_string(code: int) -> str:
    return _load().puzzle_status_string(int(code)).decode()


def puzzle_launch_count() -> int:
    return int(_load().puzzle_launch_count())


def puzzle_decode_attn_kernel_name(desc: "LayerDesc", kv: "KVView", batch: int, num_splits: int = 0) -> str:
    return _load().puzzle_decode_attn_kernel_name(ctypes.byref(desc), ctypes.byref(kv), int(batch),
                                                  int(num_splits)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise PuzzleError(code, where)


def puzzle_kv_append(desc: LayerDesc, view: KVView, k_new: torch.Tensor, v_new: torch.Tensor,
                     dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    batch = k_new.shape[0]
    _check(_load().puzzle_kv_append(ctypes.byref(desc), ctypes.byref(view), _p(k_new, torch.bfloat16, "k_new"),
                                    _p(v_new, torch.bfloat16, "v_new"), batch, _p(dev_status, torch.int32),
                                    _stream(stream)), "puzzle_kv_append")


def puzzle_kv_amax_update(x: torch.Tensor, amax: torch.Tensor, stream=None) -> None:
    """x: bf16 [n_tokens][Hkv][D] (any leading dims, flattened); amax: float32 [Hkv], raised in place."""
    hkv, d = x.shape[-2], x.shape[-1]
    n_tokens = x.numel() // (hkv * d) if x.numel() else 0
    _check(_load().puzzle_kv_amax_update(_p(x, torch.bfloat16, "x"), n_tokens, hkv, d, _p(amax, torch.float32, "amax"),
                                         _stream(stream)), "puzzle_kv_amax_update")


def puzzle_kv_scales_from_amax(amax: torch.Tensor, scale_out: torch.Tensor, pow2: bool = False, stream=None) -> None:
    _check(_load().puzzle_kv_scales_from_amax(_p(amax, torch.float32, "amax"), amax.numel(), int(bool(pow2)),
                                              _p(scale_out, torch.float32, "scale_out"), _stream(stream)),
           "puzzle_kv_scales_from_amax")


def calibrate_scales(chunks, num_kv_heads: int, pow2: bool = False, device="cuda") -> torch.Tensor:
    """Max-calibrated scales [num_kv_heads] from an iterable of bf16 tensors [..., Hkv, D] (argument
    marshalling only: one amax update per chunk, then the quotient)."""
    amax = torch.zeros(num_kv_heads, dtype=torch.float32, device=device)
    for x in chunks:
        puzzle_kv_amax_update(x, amax)
    scale = torch.empty_like(amax)
    puzzle_kv_scales_from_amax(amax, scale, pow2)
    return scale


def puzzle_kv_append_tokens(desc: LayerDesc, view: KVView, k_new: torch.Tensor, v_new: torch.Tensor,
                            new_lens: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                            stream=None) -> None:
    """k_new, v_new: bf16 [batch][n_new][Hkv][D]; new_lens: int32 [batch] or None (all n_new tokens are real)."""
    batch, n_new = k_new.shape[0], k_new.shape[1]
    _check(_load().puzzle_kv_append_tokens(ctypes.byref(desc), ctypes.byref(view), _p(k_new, torch.bfloat16, "k_new"),
                                           _p(v_new, torch.bfloat16, "v_new"), _p(new_lens, torch.int32, "new_lens"),
                                           batch, n_new, _p(dev_status, torch.int32), _stream(stream)),
           "puzzle_kv_append_tokens")


def puzzle_decode_attn_tokens_workspace_bytes(desc: LayerDesc, batch: int, n_q: int) -> int:
    return int(_load().puzzle_decode_attn_tokens_workspace_bytes(ctypes.byref(desc), int(batch), int(n_q)))


def puzzle_decode_attn_tokens_workspace_init(desc: LayerDesc, batch: int, n_q: int, workspace: torch.Tensor,
                                             stream=None) -> None:
    _check(_load().puzzle_decode_attn_tokens_workspace_init(ctypes.byref(desc), int(batch), int(n_q), _p(workspace),
                                                            workspace.numel() * workspace.element_size(),
                                                            _stream(stream)), "puzzle_decode_attn_tokens_workspace_init")


def puzzle_decode_attn_tokens(desc: LayerDesc, view: KVView, q: torch.Tensor, sinks: Optional[torch.Tensor],
                              out: torch.Tensor, lse_out: Optional[torch.Tensor] = None,
                              q_lens: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                              dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """q, out: bf16 [batch][n_q][Hq][D]; q_lens: int32 [batch] or None; see include/puzzle_attn.h."""
    if workspace is None:
        raise ValueError("a workspace tensor is required (see puzzle_decode_attn_tokens_workspace_bytes)")
    batch, n_q = q.shape[0], q.shape[1]
    _check(_load().puzzle_decode_attn_tokens(ctypes.byref(desc), ctypes.byref(view), _p(q, torch.bfloat16, "q"),
                                             _p(q_lens, torch.int32, "q_lens"), _p(sinks, torch.float32, "sinks"),
                                             _p(out, torch.bfloat16, "out"), _p(lse_out, torch.float32, "lse_out"),
                                             batch, n_q, _p(workspace), workspace.numel() * workspace.element_size(),
                                             _p(dev_status, torch.int32), _stream(stream)), "puzzle_decode_attn_tokens")


def puzzle_decode_attn_workspace_bytes(desc: LayerDesc, batch: int, num_splits: int = 0) -> int:
    return int(_load().puzzle_decode_attn_workspace_bytes(ctypes.byref(desc), int(batch), int(num_splits)))


def puzzle_decode_attn_workspace_init(desc: LayerDesc, batch: int, workspace: torch.Tensor, stream=None) -> None:
    _check(_load().puzzle_decode_attn_workspace_init(ctypes.byref(desc), int(batch), _p(workspace),
                                                     workspace.numel() * workspace.element_size(), _stream(stream)),
           "puzzle_decode_attn_workspace_init")


def _decode_attn(name: str, desc: LayerDesc, view: KVView, q, sinks, out, lse_out, num_splits, workspace, dev_status,
                 stream) -> None:
    batch = q.shape[0]
    if workspace is None:
        raise ValueError("workspace is required (size it with puzzle_decode_attn_workspace_bytes)")
    _check(getattr(_load(), name)(ctypes.byref(desc), ctypes.byref(view), _p(q, torch.bfloat16, "q"),
                                  _p(sinks, torch.float32, "sinks"), _p(out, torch.bfloat16, "out"),
                                  _p(lse_out, torch.float32, "lse_out"), batch, int(num_splits), _p(workspace),
                                  workspace.numel() * workspace.element_size(), _p(dev_status, torch.int32),
                                  _stream(stream)), name)


def puzzle_decode_attn(desc: LayerDesc, view: KVView, q: torch.Tensor, sinks: Optional[torch.Tensor],
                       out: torch.Tensor, lse_out: Optional[torch.Tensor] = None, num_splits: int = 0,
                       workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                       stream=None) -> None:
    _decode_attn("puzzle_decode_attn", desc, view, q, sinks, out, lse_out, num_splits, workspace, dev_status, stream)


def puzzle_decode_attn_tcgen05(desc: LayerDesc, view: KVView, q: torch.Tensor, sinks: Optional[torch.Tensor],
                               out: torch.Tensor, lse_out: Optional[torch.Tensor] = None, num_splits: int = 0,
                               workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                               stream=None) -> None:
    """puzzle_decode_attn computed by the tcgen05 / tensor-memory kernel (FP8 caches only)."""
    _decode_attn("puzzle_decode_attn_tcgen05", desc, view, q, sinks, out, lse_out, num_splits, workspace, dev_status,
                 stream)


def puzzle_decode_attn_static(desc: LayerDesc, view: KVView, q: torch.Tensor, sinks: Optional[torch.Tensor],
                              out: torch.Tensor, lse_out: Optional[torch.Tensor] = None, num_splits: int = 0,
                              dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """puzzle_decode_attn on the library's built-in 8 MiB scratch: for callers that cannot allocate device
    memory (no workspace tensor is involved, and nothing is allocated on the way).  Calls that share a
    device must not overlap on the GPU; make the first call on a device outside any stream capture."""
    _check(_load().puzzle_decode_attn_static(ctypes.byref(desc), ctypes.byref(view), _p(q, torch.bfloat16, "q"),
                                             _p(sinks, torch.float32, "sinks"), _p(out, torch.bfloat16, "out"),
                                             _p(lse_out, torch.float32, "lse_out"), q.shape[0], int(num_splits),
                                             _p(dev_status, torch.int32), _stream(stream)),
           "puzzle_decode_attn_static")


def puzzle_decode_step_host_staging_bytes(desc: LayerDesc, batch: int) -> int:
    return int(_load().puzzle_decode_step_host_staging_bytes(ctypes.byref(desc), int(batch)))


def _host_ptr(t: torch.Tensor, name: str):
    if t.is_cuda or not t.is_contiguous() or t.dtype != torch.bfloat16:
        raise ValueError("%s must be a contiguous bf16 host tensor" % name)
    return ctypes.c_void_p(t.data_ptr())


def puzzle_decode_step_host(desc: LayerDesc, view: KVView, q_host: torch.Tensor, k_new_host: torch.Tensor,
                            v_new_host: torch.Tensor, sinks: Optional[torch.Tensor], out_host: torch.Tensor,
                            staging: torch.Tensor, workspace: torch.Tensor, num_splits: int = 0,
                            dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """Append + attention of one layer with q, k_new, v_new and out in host memory (pinned for asynchronous copies);
    staging and workspace are device tensors.  Synchronise the stream before reading out_host."""
    _check(_load().puzzle_decode_step_host(ctypes.byref(desc), ctypes.byref(view), _host_ptr(q_host, "q_host"),
                                           _host_ptr(k_new_host, "k_new_host"), _host_ptr(v_new_host, "v_new_host"),
                                           _p(sinks, torch.float32, "sinks"), _host_ptr(out_host, "out_host"),
                                           q_host.shape[0], int(num_splits), _p(staging),
                                           staging.numel() * staging.element_size(), _p(workspace),
                                           workspace.numel() * workspace.element_size(), _p(dev_status, torch.int32),
                                           _stream(stream)), "puzzle_decode_step_host")


def puzzle_decode_attn_partial(desc: LayerDesc, view: KVView, q: torch.Tensor, o_part: torch.Tensor,
                               lse_part: torch.Tensor, num_splits: int = 0, workspace: Optional[torch.Tensor] = None,
                               dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """This device's float32 partial (o, lse) over the keys its view holds, no sink: see the header."""
    if workspace is None:
        raise ValueError("workspace is required (size it with puzzle_decode_attn_workspace_bytes)")
    _check(_load().puzzle_decode_attn_partial(ctypes.byref(desc), ctypes.byref(view), _p(q, torch.bfloat16, "q"),
                                              _p(o_part, torch.float32, "o_part"),
                                              _p(lse_part, torch.float32, "lse_part"), q.shape[0], int(num_splits),
                                              _p(workspace), workspace.numel() * workspace.element_size(),
                                              _p(dev_status, torch.int32), _stream(stream)),
           "puzzle_decode_attn_partial")


def puzzle_attn_merge_strided(part_o: torch.Tensor, part_lse: torch.Tensor, o_row_stride: int, o_part_stride: int,
                              lse_row_stride: int, lse_part_stride: int, num_parts: Optional[torch.Tensor],
                              sinks: Optional[torch.Tensor], out: torch.Tensor, num_parts_max: int,
                              lse_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """part_o / part_lse: float32 tensors whose first elements are part 0 of row 0 (strides in floats)."""
    batch, hq, d = out.shape
    _check(_load().puzzle_attn_merge_strided(_p(part_o, torch.float32, "part_o"), _p(part_lse, torch.float32, "part_lse"),
                                             int(o_row_stride), int(o_part_stride), int(lse_row_stride),
                                             int(lse_part_stride), _p(num_parts, torch.int32, "num_parts"),
                                             _p(sinks, torch.float32, "sinks"), _p(out, torch.bfloat16, "out"),
                                             _p(lse_out, torch.float32, "lse_out"), batch, hq, d, int(num_parts_max),
                                             _stream(stream)), "puzzle_attn_merge_strided")


def puzzle_attn_merge(part_o: torch.Tensor, part_lse: torch.Tensor, num_parts: Optional[torch.Tensor],
                      sinks: Optional[torch.Tensor], out: torch.Tensor, lse_out: Optional[torch.Tensor] = None,
                      stream=None) -> None:
    batch, hq, s, d = part_o.shape
    _check(_load().puzzle_attn_merge(_p(part_o, torch.float32, "part_o"), _p(part_lse, torch.float32, "part_lse"),
                                     _p(num_parts, torch.int32, "num_parts"), _p(sinks, torch.float32, "sinks"),
                                     _p(out, torch.bfloat16, "out"), _p(lse_out, torch.float32, "lse_out"),
                                     batch, hq, d, s, _stream(stream)), "puzzle_attn_merge")


def puzzle_hbm_read_probe(buf: torch.Tensor, sink: torch.Tensor, stream=None) -> None:
    _check(_load().puzzle_hbm_read_probe(_p(buf), buf.numel() * buf.element_size(), _p(sink), _stream(stream)),
           "puzzle_hbm_read_probe")
