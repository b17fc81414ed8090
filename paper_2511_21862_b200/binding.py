"""ctypes binding of the `ooco_*` C ABI: argument marshalling only.

Every function takes torch tensors (device memory owned by the caller), passes their raw
pointers through the C boundary and raises `OocoError` on a non-zero status.  There is no
fallback: without the built CUDA library the import of the library fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libooco.so")

EXPORTS = (
    "ooco_kv_append", "ooco_decode_workspace_bytes", "ooco_decode_attention", "ooco_workspace_status",
    "ooco_decode_bytes_model", "ooco_step_staging_bytes", "ooco_decode_step_host", "ooco_decode_step",
    "ooco_last_launch_count", "ooco_last_error_detail", "ooco_set_tuning", "ooco_status_string", "ooco_version",
    "ooco_profile_enable", "ooco_profile_read", "ooco_decode_attention_static",
    "ooco_kv_gather_blocks", "ooco_kv_scatter_blocks", "ooco_kv_copy_blocks",
    "ooco_kv_append_fp8", "ooco_decode_attention_fp8", "ooco_decode_step_fp8",
    "ooco_decode_workspace_bytes_mq", "ooco_decode_attention_mq", "ooco_kv_append_mq", "ooco_attention_bytes_model",
    "ooco_decode_step_mq", "ooco_decode_step_mq_fp8", "ooco_get_tuning", "ooco_checked_build", "ooco_check_predicate",
    "ooco_last_host_step_ns",
)


class OocoError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = lib().ooco_last_error_detail().decode() if status in (-4, -5) else ""
        super().__init__(f"{where}: {status_string(status)} ({status}) {detail}".rstrip())


class ooco_shape_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch", "num_q_heads", "num_kv_heads", "head_dim", "block_size", "num_blocks",
        "max_blocks_per_seq", "reserved")] + [(n, ctypes.c_int64) for n in (
            "kv_block_stride", "kv_head_stride", "kv_token_stride")]


class ooco_cost_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "flops", "bytes_q", "bytes_out", "bytes_kv", "bytes_index", "bytes_paper", "total_tokens")]


_lib = None


def use_library(path: str | None):
    """Makes `path` (e.g. the checked build, `build.LIB_CHECKED`) the library every call below goes to;
    None returns to the default library.  Returns the path that was in use."""
    global _lib, LIB_PATH
    old = LIB_PATH
    LIB_PATH = path or os.path.join(_HERE, "libooco.so")
    _lib = None
    lib()
    return old


def lib() -> ctypes.CDLL:
    """The loaded shared library (built by `paper_2511_21862_b200.build`); no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2511_21862_b200.build` "
                              "(there is no non-CUDA fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32p = ctypes.c_void_p, ctypes.c_void_p
        sp = ctypes.POINTER(ooco_shape_t)
        L.ooco_kv_append.restype = ctypes.c_int
        L.ooco_kv_append.argtypes = [sp, vp, vp, vp, vp, i32p, i32p, vp]
        L.ooco_decode_workspace_bytes.restype = ctypes.c_size_t
        L.ooco_decode_workspace_bytes.argtypes = [sp]
        L.ooco_decode_attention.restype = ctypes.c_int
        L.ooco_decode_attention.argtypes = [sp, vp, vp, vp, i32p, i32p, ctypes.c_float, vp, vp,
                                            ctypes.c_size_t, vp]
        L.ooco_decode_step.restype = ctypes.c_int
        L.ooco_decode_step.argtypes = [sp, vp, vp, vp, vp, vp, i32p, i32p, i32p, ctypes.c_float, vp, vp,
                                       ctypes.c_size_t, vp]
        L.ooco_decode_attention_static.restype = ctypes.c_int
        L.ooco_decode_attention_static.argtypes = [sp, vp, vp, vp, i32p, i32p, ctypes.c_float, vp, vp]
        f32 = ctypes.c_float
        L.ooco_kv_append_fp8.restype = ctypes.c_int
        L.ooco_kv_append_fp8.argtypes = [sp, vp, vp, vp, vp, i32p, i32p, f32, f32, vp]
        L.ooco_decode_attention_fp8.restype = ctypes.c_int
        L.ooco_decode_attention_fp8.argtypes = [sp, vp, vp, vp, i32p, i32p, f32, f32, f32, vp, vp, ctypes.c_size_t, vp]
        L.ooco_decode_step_fp8.restype = ctypes.c_int
        L.ooco_decode_step_fp8.argtypes = [sp, vp, vp, vp, vp, vp, i32p, i32p, i32p, f32, f32, f32, vp, vp,
                                           ctypes.c_size_t, vp]
        L.ooco_decode_workspace_bytes_mq.restype = ctypes.c_size_t
        L.ooco_decode_workspace_bytes_mq.argtypes = [sp, ctypes.c_int32]
        L.ooco_decode_attention_mq.restype = ctypes.c_int
        L.ooco_decode_attention_mq.argtypes = [sp, ctypes.c_int32, vp, vp, vp, i32p, i32p, ctypes.c_float, vp, vp,
                                               ctypes.c_size_t, vp]
        L.ooco_decode_step_mq.restype = ctypes.c_int
        L.ooco_decode_step_mq.argtypes = [sp, ctypes.c_int32, vp, vp, vp, vp, vp, i32p, i32p, i32p, ctypes.c_float, vp,
                                          vp, ctypes.c_size_t, vp]
        L.ooco_decode_step_mq_fp8.restype = ctypes.c_int
        L.ooco_decode_step_mq_fp8.argtypes = [sp, ctypes.c_int32, vp, vp, vp, vp, vp, i32p, i32p, i32p, ctypes.c_float,
                                              ctypes.c_float, ctypes.c_float, vp, vp, ctypes.c_size_t, vp]
        L.ooco_kv_append_mq.restype = ctypes.c_int
        L.ooco_kv_append_mq.argtypes = [sp, ctypes.c_int32, vp, vp, vp, vp, i32p, i32p, vp]
        L.ooco_kv_gather_blocks.restype = ctypes.c_int
        L.ooco_kv_gather_blocks.argtypes = [sp, vp, vp, i32p, ctypes.c_int32, vp, vp, i32p, vp]
        L.ooco_kv_scatter_blocks.restype = ctypes.c_int
        L.ooco_kv_scatter_blocks.argtypes = [sp, vp, vp, i32p, ctypes.c_int32, vp, vp, i32p, vp]
        L.ooco_kv_copy_blocks.restype = ctypes.c_int
        L.ooco_kv_copy_blocks.argtypes = [sp, vp, vp, i32p, i32p, ctypes.c_int32, i32p, vp]
        L.ooco_workspace_status.restype = ctypes.c_int
        L.ooco_workspace_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
        L.ooco_decode_bytes_model.restype = ctypes.c_int
        L.ooco_decode_bytes_model.argtypes = [sp, i32p, ctypes.c_int32, ctypes.POINTER(ooco_cost_t)]
        L.ooco_attention_bytes_model.restype = ctypes.c_int
        L.ooco_attention_bytes_model.argtypes = [sp, ctypes.c_int32, i32p, ctypes.c_int32, ctypes.POINTER(ooco_cost_t)]
        L.ooco_step_staging_bytes.restype = ctypes.c_size_t
        L.ooco_step_staging_bytes.argtypes = [sp]
        L.ooco_decode_step_host.restype = ctypes.c_int
        L.ooco_decode_step_host.argtypes = [sp, vp, vp, vp, i32p, i32p, i32p, vp, vp, ctypes.c_float, vp,
                                            vp, ctypes.c_size_t, vp, ctypes.c_size_t, vp]
        L.ooco_last_launch_count.restype = ctypes.c_int
        L.ooco_last_error_detail.restype = ctypes.c_char_p
        L.ooco_set_tuning.restype = ctypes.c_int
        L.ooco_set_tuning.argtypes = [ctypes.c_int, ctypes.c_int]
        L.ooco_get_tuning.restype = ctypes.c_int
        L.ooco_get_tuning.argtypes = [ctypes.c_int]
        L.ooco_last_host_step_ns.restype = ctypes.c_int
        L.ooco_last_host_step_ns.argtypes = [ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]
        L.ooco_checked_build.restype = ctypes.c_int
        L.ooco_check_predicate.restype = ctypes.c_int
        L.ooco_check_predicate.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        L.ooco_status_string.restype = ctypes.c_char_p
        L.ooco_status_string.argtypes = [ctypes.c_int]
        L.ooco_version.restype = ctypes.c_int
        L.ooco_profile_enable.restype = ctypes.c_int
        L.ooco_profile_enable.argtypes = [ctypes.c_int]
        L.ooco_profile_read.restype = ctypes.c_int
        L.ooco_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().ooco_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise OocoError(status, where)


@dataclass(frozen=True)
class Shape:
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    num_blocks: int
    max_blocks_per_seq: int
    kv_block_stride: int
    kv_head_stride: int
    kv_token_stride: int

    def c(self) -> ooco_shape_t:
        return ooco_shape_t(self.batch, self.num_q_heads, self.num_kv_heads, self.head_dim, self.block_size,
                            self.num_blocks, self.max_blocks_per_seq, 0, self.kv_block_stride,
                            self.kv_head_stride, self.kv_token_stride)


KNOBS = {"warps": 0, "stages": 1, "ctas_per_sm": 2, "chunk_min": 3, "chunk_max": 4, "items_per_cta": 5,
         "split_halves": 6, "tiles_per_warp": 7, "pdl": 8, "copy_ctas_per_sm": 9, "host_stage_kernel": 10, "row_layout_16": 11, "chunk_tcgen05": 12,
         "out_f32": 13, "kv8_tcgen05": 14, "chunk_two_tiles": 15}


def set_tuning(**kw):
    for k, v in kw.items():
        _check(lib().ooco_set_tuning(KNOBS[k], int(v)), f"ooco_set_tuning({k}={v})")


def get_tuning(knob: str) -> int:
    v = lib().ooco_get_tuning(KNOBS[knob])
    if v < 0:
        raise OocoError(v, f"ooco_get_tuning({knob})")
    return int(v)


def last_host_step_ns():
    """(ns until everything of the last decode_step_host call was enqueued, ns it then waited for the stream)."""
    a, b = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(lib().ooco_last_host_step_ns(ctypes.byref(a), ctypes.byref(b)), "ooco_last_host_step_ns")
    return int(a.value), int(b.value)


def checked_build() -> bool:
    """True when the loaded library is the variant whose kernels range-check device-derived indices."""
    return bool(lib().ooco_checked_build())


def check_predicate(which: int, *args) -> bool:
    """Host evaluation of one of the checked build's range predicates (see ooco_check_predicate)."""
    a = (ctypes.c_int64 * max(1, len(args)))(*[int(x) for x in args])
    r = lib().ooco_check_predicate(int(which), a)
    if r < 0:
        raise OocoError(r, "ooco_check_predicate")
    return bool(r)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev(t: torch.Tensor, dtype=None) -> int:
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t.data_ptr()


def _out(t: torch.Tensor) -> int:
    """`out` is bf16, or fp32 while the diagnostic fp32-output knob is set."""
    want = torch.float32 if get_tuning("out_f32") else torch.bfloat16
    return _dev(t, want)


def workspace_bytes(shape: Shape) -> int:
    n = lib().ooco_decode_workspace_bytes(ctypes.byref(shape.c()))
    if n == 0:
        raise OocoError(-3, "ooco_decode_workspace_bytes")
    return int(n)


def step_staging_bytes(shape: Shape) -> int:
    n = lib().ooco_step_staging_bytes(ctypes.byref(shape.c()))
    if n == 0:
        raise OocoError(-3, "ooco_step_staging_bytes")
    return int(n)


def kv_append(shape: Shape, k_new, v_new, k_cache, v_cache, block_table, positions, stream=None):
    _check(lib().ooco_kv_append(
        ctypes.byref(shape.c()), _dev(k_new, torch.bfloat16), _dev(v_new, torch.bfloat16),
        _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16), _dev(block_table, torch.int32),
        _dev(positions, torch.int32), _stream_ptr(stream)), "ooco_kv_append")


def decode_attention(shape: Shape, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace,
                     stream=None):
    _check(lib().ooco_decode_attention(
        ctypes.byref(shape.c()), _dev(q, torch.bfloat16), _dev(k_cache, torch.bfloat16),
        _dev(v_cache, torch.bfloat16), _dev(block_table, torch.int32), _dev(context_lens, torch.int32),
        float(scale), _out(out), _dev(workspace), workspace.numel() * workspace.element_size(),
        _stream_ptr(stream)), "ooco_decode_attention")


def decode_step(shape: Shape, q, k_new, v_new, k_cache, v_cache, block_table, positions, context_lens, scale, out,
                workspace, stream=None):
    """Fused append (at `positions`) + attention (over `context_lens`) on device buffers."""
    _check(lib().ooco_decode_step(
        ctypes.byref(shape.c()), _dev(q, torch.bfloat16), _dev(k_new, torch.bfloat16), _dev(v_new, torch.bfloat16),
        _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16), _dev(block_table, torch.int32),
        _dev(positions, torch.int32), _dev(context_lens, torch.int32), float(scale), _out(out),
        _dev(workspace), workspace.numel() * workspace.element_size(), _stream_ptr(stream)), "ooco_decode_step")


def kv_append_fp8(shape: Shape, k_new, v_new, k_cache, v_cache, block_table, positions, k_scale, v_scale,
                  stream=None):
    """Quantising append into uint8 (E4M3) caches."""
    _check(lib().ooco_kv_append_fp8(
        ctypes.byref(shape.c()), _dev(k_new, torch.bfloat16), _dev(v_new, torch.bfloat16),
        _dev(k_cache, torch.uint8), _dev(v_cache, torch.uint8), _dev(block_table, torch.int32),
        _dev(positions, torch.int32), float(k_scale), float(v_scale), _stream_ptr(stream)), "ooco_kv_append_fp8")


def decode_attention_fp8(shape: Shape, q, k_cache, v_cache, block_table, context_lens, scale, k_scale, v_scale, out,
                         workspace, stream=None):
    """Decode attention over uint8 (E4M3) caches; q / out bf16."""
    _check(lib().ooco_decode_attention_fp8(
        ctypes.byref(shape.c()), _dev(q, torch.bfloat16), _dev(k_cache, torch.uint8), _dev(v_cache, torch.uint8),
        _dev(block_table, torch.int32), _dev(context_lens, torch.int32), float(scale), float(k_scale),
        float(v_scale), _out(out), _dev(workspace), workspace.numel() * workspace.element_size(),
        _stream_ptr(stream)), "ooco_decode_attention_fp8")


def decode_step_fp8(shape: Shape, q, k_new, v_new, k_cache, v_cache, block_table, positions, context_lens, scale,
                    k_scale, v_scale, out, workspace, stream=None):
    """Fused quantising append + attention over uint8 (E4M3) caches."""
    _check(lib().ooco_decode_step_fp8(
        ctypes.byref(shape.c()), _dev(q, torch.bfloat16), _dev(k_new, torch.bfloat16), _dev(v_new, torch.bfloat16),
        _dev(k_cache, torch.uint8), _dev(v_cache, torch.uint8), _dev(block_table, torch.int32),
        _dev(positions, torch.int32), _dev(context_lens, torch.int32), float(scale), float(k_scale), float(v_scale),
        _out(out), _dev(workspace), workspace.numel() * workspace.element_size(),
        _stream_ptr(stream)), "ooco_decode_step_fp8")


def workspace_bytes_mq(shape: Shape, q_len: int) -> int:
    n = lib().ooco_decode_workspace_bytes_mq(ctypes.byref(shape.c()), int(q_len))
    if n == 0:
        raise OocoError(-3, "ooco_decode_workspace_bytes_mq")
    return int(n)


def decode_attention_mq(shape: Shape, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace,
                        stream=None):
    """q, out: bf16 [B, q_len, Hq, D]; the query tokens are the last q_len tokens of each context."""
    assert q.dim() == 4 and q.shape == out.shape
    _check(lib().ooco_decode_attention_mq(
        ctypes.byref(shape.c()), int(q.shape[1]), _dev(q, torch.bfloat16), _dev(k_cache, torch.bfloat16),
        _dev(v_cache, torch.bfloat16), _dev(block_table, torch.int32), _dev(context_lens, torch.int32),
        float(scale), _out(out), _dev(workspace), workspace.numel() * workspace.element_size(),
        _stream_ptr(stream)), "ooco_decode_attention_mq")


def decode_step_mq(shape: Shape, q, k_new, v_new, k_cache, v_cache, block_table, positions, context_lens, scale, out,
                   workspace, stream=None):
    """Fused append of q_len new tokens (at positions[b] + i) + causal attention over context_lens."""
    assert q.dim() == 4 and q.shape == out.shape and k_new.shape[1] == q.shape[1]
    _check(lib().ooco_decode_step_mq(
        ctypes.byref(shape.c()), int(q.shape[1]), _dev(q, torch.bfloat16), _dev(k_new, torch.bfloat16),
        _dev(v_new, torch.bfloat16), _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16),
        _dev(block_table, torch.int32), _dev(positions, torch.int32), _dev(context_lens, torch.int32), float(scale),
        _out(out), _dev(workspace), workspace.numel() * workspace.element_size(),
        _stream_ptr(stream)), "ooco_decode_step_mq")


def decode_step_mq_fp8(shape: Shape, q, k_new, v_new, k_cache, v_cache, block_table, positions, context_lens, scale,
                       k_scale, v_scale, out, workspace, stream=None):
    """Several query tokens over uint8 (E4M3) caches; k_new = v_new = None runs the attention only."""
    assert q.dim() == 4 and q.shape == out.shape
    _check(lib().ooco_decode_step_mq_fp8(
        ctypes.byref(shape.c()), int(q.shape[1]), _dev(q, torch.bfloat16), _opt_dev(k_new, torch.bfloat16),
        _opt_dev(v_new, torch.bfloat16), _dev(k_cache, torch.uint8), _dev(v_cache, torch.uint8),
        _dev(block_table, torch.int32), _opt_dev(positions, torch.int32), _dev(context_lens, torch.int32),
        float(scale), float(k_scale), float(v_scale), _out(out), _dev(workspace),
        workspace.numel() * workspace.element_size(), _stream_ptr(stream)), "ooco_decode_step_mq_fp8")


def kv_append_mq(shape: Shape, k_new, v_new, k_cache, v_cache, block_table, positions, stream=None):
    """k_new, v_new: bf16 [B, q_len, Hkv, D]; token i of sequence b goes to position positions[b] + i."""
    assert k_new.dim() == 4 and k_new.shape == v_new.shape
    _check(lib().ooco_kv_append_mq(
        ctypes.byref(shape.c()), int(k_new.shape[1]), _dev(k_new, torch.bfloat16), _dev(v_new, torch.bfloat16),
        _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16), _dev(block_table, torch.int32),
        _dev(positions, torch.int32), _stream_ptr(stream)), "ooco_kv_append_mq")


STATIC_SCRATCH_BYTES = 16 << 20


def decode_attention_static(shape: Shape, q, k_cache, v_cache, block_table, context_lens, scale, out, stream=None):
    """ooco_decode_attention without a workspace argument, for callers that cannot allocate device
    memory (the whole device already belongs to a KV pool, an allocation's implicit synchronisation is
    not affordable, or the host framework forbids allocations outside its pool).  The scratch is a
    16 MiB array built into the library; shapes that need more raise OocoError(-4).  Calls that may
    overlap on the GPU race on that array; the first call on a device should precede stream capture."""
    _check(lib().ooco_decode_attention_static(
        ctypes.byref(shape.c()), _dev(q, torch.bfloat16), _dev(k_cache, torch.bfloat16),
        _dev(v_cache, torch.bfloat16), _dev(block_table, torch.int32), _dev(context_lens, torch.int32),
        float(scale), _out(out), _stream_ptr(stream)), "ooco_decode_attention_static")


def _opt_dev(t, dtype=None):
    return None if t is None else _dev(t, dtype)


def kv_gather_blocks(shape: Shape, k_cache, v_cache, block_ids, k_packed, v_packed, status=None, stream=None):
    """Pack the listed pool blocks, in list order, into `k_packed` / `v_packed` [n, Hkv, bs, D]."""
    n = block_ids.numel()
    need = n * shape.num_kv_heads * shape.block_size * shape.head_dim
    assert k_packed.numel() >= need and v_packed.numel() >= need
    _check(lib().ooco_kv_gather_blocks(
        ctypes.byref(shape.c()), _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16),
        _dev(block_ids, torch.int32), n, _dev(k_packed, torch.bfloat16), _dev(v_packed, torch.bfloat16),
        _opt_dev(status, torch.int32), _stream_ptr(stream)), "ooco_kv_gather_blocks")


def kv_scatter_blocks(shape: Shape, k_packed, v_packed, block_ids, k_cache, v_cache, status=None, stream=None):
    """Write block i of the packed buffers to pool block `block_ids[i]`."""
    n = block_ids.numel()
    need = n * shape.num_kv_heads * shape.block_size * shape.head_dim
    assert k_packed.numel() >= need and v_packed.numel() >= need
    _check(lib().ooco_kv_scatter_blocks(
        ctypes.byref(shape.c()), _dev(k_packed, torch.bfloat16), _dev(v_packed, torch.bfloat16),
        _dev(block_ids, torch.int32), n, _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16),
        _opt_dev(status, torch.int32), _stream_ptr(stream)), "ooco_kv_scatter_blocks")


def kv_copy_blocks(shape: Shape, k_cache, v_cache, src_ids, dst_ids, status=None, stream=None):
    """Copy pool block `src_ids[i]` to pool block `dst_ids[i]`."""
    n = src_ids.numel()
    assert dst_ids.numel() == n
    _check(lib().ooco_kv_copy_blocks(
        ctypes.byref(shape.c()), _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16),
        _dev(src_ids, torch.int32), _dev(dst_ids, torch.int32), n, _opt_dev(status, torch.int32),
        _stream_ptr(stream)), "ooco_kv_copy_blocks")


def workspace_status(workspace, stream=None) -> int:
    """Synchronises the stream and returns the device status word (0 = clean)."""
    v = ctypes.c_int32(0)
    rc = lib().ooco_workspace_status(_dev(workspace), _stream_ptr(stream), ctypes.byref(v))
    if rc not in (0, -6):
        raise OocoError(rc, "ooco_workspace_status")
    return int(v.value)


def decode_bytes_model(shape: Shape, context_lens_host, bytes_per_value: int = 2) -> dict:
    """Host-only: `context_lens_host` is a CPU int32 tensor."""
    t = context_lens_host
    assert not t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()
    c = ooco_cost_t()
    _check(lib().ooco_decode_bytes_model(ctypes.byref(shape.c()), t.data_ptr(), bytes_per_value,
                                         ctypes.byref(c)), "ooco_decode_bytes_model")
    return {n: int(getattr(c, n)) for n, _ in ooco_cost_t._fields_}


def attention_bytes_model(shape: Shape, q_len: int, context_lens_host, bytes_per_value: int = 2) -> dict:
    """Host-only: the operator table's attention row with S_q = q_len."""
    t = context_lens_host
    assert not t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()
    c = ooco_cost_t()
    _check(lib().ooco_attention_bytes_model(ctypes.byref(shape.c()), int(q_len), t.data_ptr(), bytes_per_value,
                                            ctypes.byref(c)), "ooco_attention_bytes_model")
    return {n: int(getattr(c, n)) for n, _ in ooco_cost_t._fields_}


def decode_step_host(shape: Shape, q_host, k_new_host, v_new_host, block_table_host, positions_host,
                     context_lens_host, k_cache, v_cache, scale, out_host, staging, workspace, stream=None):
    """One append + attention step from host (ideally pinned) buffers; returns with out_host filled."""
    for t in (q_host, k_new_host, v_new_host, block_table_host, positions_host, context_lens_host, out_host):
        assert not t.is_cuda and t.is_contiguous()
    _check(lib().ooco_decode_step_host(
        ctypes.byref(shape.c()), q_host.data_ptr(), k_new_host.data_ptr(), v_new_host.data_ptr(),
        block_table_host.data_ptr(), positions_host.data_ptr(), context_lens_host.data_ptr(),
        _dev(k_cache, torch.bfloat16), _dev(v_cache, torch.bfloat16), float(scale), out_host.data_ptr(),
        _dev(staging), staging.numel() * staging.element_size(), _dev(workspace),
        workspace.numel() * workspace.element_size(), _stream_ptr(stream)), "ooco_decode_step_host")


def profile_enable(max_records: int):
    _check(lib().ooco_profile_enable(int(max_records)), "ooco_profile_enable")


def profile_read(max_records: int):
    """[(plan_ms, attention_ms, merge_ms), ...] of the calls recorded since the last read."""
    buf = (ctypes.c_float * (3 * max_records))()
    n = ctypes.c_int(0)
    _check(lib().ooco_profile_read(buf, max_records, ctypes.byref(n)), "ooco_profile_read")
    return [(buf[3 * i], buf[3 * i + 1], buf[3 * i + 2]) for i in range(n.value)]


def last_launch_count() -> int:
    return int(lib().ooco_last_launch_count())


def shape_of(batch) -> Shape:
    """Shape struct of a `paper_2511_21862_b200.inputs.DecodeBatch`."""
    cfg = batch.cfg
    bstr, hstr, tstr = batch.strides
    return Shape(batch.context_lens.numel(), cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.block_size,
                 batch.num_blocks, batch.max_blocks_per_seq, bstr, hstr, tstr)
