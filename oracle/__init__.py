"""fp64 CPU oracle of the paged decode path (TEST INFRASTRUCTURE ONLY).

Thin ctypes/numpy access to ``ooco_oracle.c``.  Only the tests, the smoke check
and the benchmark's CPU-baseline / reference legs may import this package; the
product package never does, and nothing here imports the product package.
bf16 tensors are exchanged as ``numpy.uint16`` arrays of the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, "ooco_oracle.c"), os.path.join(_HERE, "ooco_oracle_fp8.c")]
_LIB_PATH = os.path.join(_HERE, "libooco_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ooco_oracle.c with gcc (OpenMP, no fast-math) next to its source."""
    stale = (not os.path.exists(_LIB_PATH)) or any(os.path.getmtime(_LIB_PATH) < os.path.getmtime(s) for s in _SRCS)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC",
               "-o", _LIB_PATH] + _SRCS + ["-lm"]
        subprocess.run(cmd, check=True)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, f64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_decode_attention.restype = ctypes.c_int
        lib.oracle_decode_attention.argtypes = [i32] * 7 + [i64] * 3 + [vp] * 5 + [f64, vp, i64, vp, vp, vp]
        lib.oracle_kv_append.restype = i64
        lib.oracle_kv_append.argtypes = [i32] * 6 + [i64] * 3 + [vp] * 6
        lib.oracle_bytes_model.restype = ctypes.c_int
        lib.oracle_bytes_model.argtypes = [i32] * 5 + [vp, i32, vp]
        lib.oracle_num_threads.restype = ctypes.c_int
        f32, u8 = ctypes.c_float, ctypes.c_uint8
        lib.oracle_e4m3_decode.restype = f64
        lib.oracle_e4m3_decode.argtypes = [u8]
        lib.oracle_e4m3_encode.restype = u8
        lib.oracle_e4m3_encode.argtypes = [f32]
        lib.oracle_decode_attention_fp8.restype = ctypes.c_int
        lib.oracle_decode_attention_fp8.argtypes = [i32] * 7 + [i64] * 3 + [vp] * 5 + [f64, f32, f32, vp, i64, vp, vp, vp]
        lib.oracle_kv_append_fp8.restype = i64
        lib.oracle_kv_append_fp8.argtypes = [i32] * 6 + [i64] * 3 + [vp] * 6 + [f32, f32]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the attention oracle uses (OpenMP's maximum)."""
    return int(_load().oracle_num_threads())


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


@dataclass
class AttentionResult:
    out: np.ndarray   # float64 [B, Hq, D]
    lse: np.ndarray   # float64 [B, Hq], natural-log-sum-exp of the scaled scores
    wsum: np.ndarray  # float64 [B, Hq], sum of the softmax weights


def decode_attention(q, k_cache, v_cache, block_table, context_lens, scale, *, num_kv_heads,
                     block_size, strides, pairs=None) -> AttentionResult:
    """Softmax attention of one query token per sequence over its paged KV cache.

    q: uint16 [B, Hq, D]; k_cache / v_cache: flat or shaped uint16 pools addressed through
    ``strides`` = (block, head, token) element strides; block_table: int32 [B, MB];
    context_lens: int32 [B]; pairs: optional int32 [n, 2] list of (b, hq) rows to compute
    (all other rows of the result are NaN).
    """
    lib = _load()
    q = _u16(q)
    B, Hq, D = q.shape
    k_cache, v_cache = _u16(k_cache), _u16(v_cache)
    block_table, context_lens = _i32(block_table), _i32(context_lens)
    assert block_table.ndim == 2 and block_table.shape[0] == B and context_lens.shape == (B,)
    MB = block_table.shape[1]
    bstr, hstr, tstr = (int(s) for s in strides)
    num_blocks = k_cache.size // bstr
    assert k_cache.size == v_cache.size
    out = np.full((B, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    wsum = np.full((B, Hq), np.nan, dtype=np.float64)
    if pairs is not None:
        pairs = _i32(pairs).reshape(-1, 2)
        pp, npairs = _ptr(pairs), pairs.shape[0]
    else:
        pp, npairs = None, 0
    rc = lib.oracle_decode_attention(B, Hq, num_kv_heads, D, block_size, num_blocks, MB, bstr, hstr,
                                     tstr, _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                     _ptr(context_lens), float(scale), pp, npairs, _ptr(out),
                                     _ptr(lse), _ptr(wsum))
    if rc != 0:
        raise ValueError(f"oracle_decode_attention failed with {rc}")
    return AttentionResult(out, lse, wsum)


def decode_attention_mq(q, k_cache, v_cache, block_table, context_lens, scale, *, num_kv_heads, block_size,
                        strides) -> AttentionResult:
    """Several query tokens per sequence (the operator table's S_q > 1: multi-token decode, a chunk of
    a prefill): q is uint16 [B, Sq, Hq, D], the Sq query tokens are the LAST Sq tokens of the sequence,
    context_lens[b] counts them, and query i sees tokens [0, T_b - Sq + i + 1) -- causal attention over the
    cache.  By definition this is the one-query operator on B * Sq rows with those lengths, which is how
    it is computed.  Results are shaped [B, Sq, Hq, ...]; a query without visible tokens gives zeros."""
    q = _u16(q)
    B, Sq, Hq, D = q.shape
    lens = _i32(context_lens)
    table = _i32(block_table)
    lens_x = (lens[:, None] - Sq + 1 + np.arange(Sq, dtype=np.int32)[None, :]).reshape(-1)
    lens_x = np.where(np.repeat(lens, Sq) <= 0, 0, np.maximum(lens_x, 0)).astype(np.int32)
    table_x = np.repeat(table, Sq, axis=0)
    r = decode_attention(q.reshape(B * Sq, Hq, D), k_cache, v_cache, table_x, lens_x, scale,
                         num_kv_heads=num_kv_heads, block_size=block_size, strides=strides)
    return AttentionResult(r.out.reshape(B, Sq, Hq, D), r.lse.reshape(B, Sq, Hq), r.wsum.reshape(B, Sq, Hq))


def kv_append(k_new, v_new, k_cache, v_cache, block_table, positions, *, block_size, strides) -> int:
    """In-place append of k_new / v_new uint16 [B, Hkv, D] into the uint16 pools. Returns rows written."""
    lib = _load()
    k_new, v_new = _u16(k_new), _u16(v_new)
    B, Hkv, D = k_new.shape
    assert k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16
    assert k_cache.flags.c_contiguous and v_cache.flags.c_contiguous and k_cache.flags.writeable
    block_table, positions = _i32(block_table), _i32(positions)
    MB = block_table.shape[1]
    bstr, hstr, tstr = (int(s) for s in strides)
    num_blocks = k_cache.size // bstr
    return int(lib.oracle_kv_append(B, Hkv, D, block_size, num_blocks, MB, bstr, hstr, tstr,
                                    _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache),
                                    _ptr(block_table), _ptr(positions)))


# --------------------------------------------------------------------------- 8-bit (E4M3) KV cache
def e4m3_decode(codes) -> np.ndarray:
    """float64 values of E4M3 codes (uint8), from the format's definition."""
    lib = _load()
    codes = np.asarray(codes, dtype=np.uint8)
    return np.array([lib.oracle_e4m3_decode(int(c)) for c in codes.reshape(-1)], dtype=np.float64).reshape(codes.shape)


def e4m3_encode(values) -> np.ndarray:
    """Nearest-even, saturating E4M3 codes of float32 values."""
    lib = _load()
    values = np.asarray(values, dtype=np.float32)
    return np.array([lib.oracle_e4m3_encode(float(x)) for x in values.reshape(-1)], dtype=np.uint8).reshape(values.shape)


def _u8(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint8, a.dtype
    return a


def decode_attention_fp8(q, k_cache, v_cache, block_table, context_lens, scale, k_scale, v_scale, *, num_kv_heads,
                         block_size, strides, pairs=None) -> AttentionResult:
    """decode_attention over uint8 E4M3 pools; a stored code stands for decode(code) * k_scale (v_scale)."""
    lib = _load()
    q = _u16(q)
    B, Hq, D = q.shape
    k_cache, v_cache = _u8(k_cache), _u8(v_cache)
    block_table, context_lens = _i32(block_table), _i32(context_lens)
    MB = block_table.shape[1]
    bstr, hstr, tstr = (int(s) for s in strides)
    num_blocks = k_cache.size // bstr
    out = np.full((B, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    wsum = np.full((B, Hq), np.nan, dtype=np.float64)
    if pairs is not None:
        pairs = _i32(pairs).reshape(-1, 2)
        pp, npairs = _ptr(pairs), pairs.shape[0]
    else:
        pp, npairs = None, 0
    rc = lib.oracle_decode_attention_fp8(B, Hq, num_kv_heads, D, block_size, num_blocks, MB, bstr, hstr, tstr,
                                         _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                         _ptr(context_lens), float(scale), float(k_scale), float(v_scale), pp,
                                         npairs, _ptr(out), _ptr(lse), _ptr(wsum))
    if rc != 0:
        raise ValueError(f"oracle_decode_attention_fp8 failed with {rc}")
    return AttentionResult(out, lse, wsum)


def decode_attention_mq_fp8(q, k_cache, v_cache, block_table, context_lens, scale, k_scale, v_scale, *, num_kv_heads,
                            block_size, strides) -> AttentionResult:
    """decode_attention_mq over uint8 E4M3 pools: the one-query 8-bit operator on B * Sq rows."""
    q = _u16(q)
    B, Sq, Hq, D = q.shape
    lens = _i32(context_lens)
    lens_x = (lens[:, None] - Sq + 1 + np.arange(Sq, dtype=np.int32)[None, :]).reshape(-1)
    lens_x = np.where(np.repeat(lens, Sq) <= 0, 0, np.maximum(lens_x, 0)).astype(np.int32)
    r = decode_attention_fp8(q.reshape(B * Sq, Hq, D), k_cache, v_cache, np.repeat(_i32(block_table), Sq, axis=0),
                             lens_x, scale, k_scale, v_scale, num_kv_heads=num_kv_heads, block_size=block_size,
                             strides=strides)
    return AttentionResult(r.out.reshape(B, Sq, Hq, D), r.lse.reshape(B, Sq, Hq), r.wsum.reshape(B, Sq, Hq))


def kv_append_fp8(k_new, v_new, k_cache, v_cache, block_table, positions, k_scale, v_scale, *, block_size,
                  strides) -> int:
    """In-place quantising append of bf16 rows (uint16 bits) into uint8 E4M3 pools."""
    lib = _load()
    k_new, v_new = _u16(k_new), _u16(v_new)
    B, Hkv, D = k_new.shape
    assert k_cache.dtype == np.uint8 and v_cache.dtype == np.uint8
    assert k_cache.flags.c_contiguous and v_cache.flags.c_contiguous and k_cache.flags.writeable
    block_table, positions = _i32(block_table), _i32(positions)
    MB = block_table.shape[1]
    bstr, hstr, tstr = (int(s) for s in strides)
    num_blocks = k_cache.size // bstr
    return int(lib.oracle_kv_append_fp8(B, Hkv, D, block_size, num_blocks, MB, bstr, hstr, tstr, _ptr(k_new),
                                        _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(block_table),
                                        _ptr(positions), float(k_scale), float(v_scale)))


COST_FIELDS = ("flops", "bytes_q", "bytes_out", "bytes_kv", "bytes_index", "bytes_paper", "total_tokens")


def bytes_model(context_lens, *, num_q_heads, num_kv_heads, head_dim, block_size, bytes_per_value=2) -> dict:
    """Attention row of the paper's operator table summed over the batch, as a dict of ints."""
    lib = _load()
    context_lens = _i32(context_lens)
    cost = np.zeros(7, dtype=np.int64)
    rc = lib.oracle_bytes_model(context_lens.shape[0], num_q_heads, num_kv_heads, head_dim, block_size,
                                _ptr(context_lens), bytes_per_value, _ptr(cost))
    if rc != 0:
        raise ValueError(f"oracle_bytes_model failed with {rc}")
    return {k: int(v) for k, v in zip(COST_FIELDS, cost)}


# --------------------------------------------------------------------------- paged block movement
# Migration of an offline request moves its KV cache between instances (section 3.4.3 of the
# paper, "Offline Request Migration"; section 4: the KV cache is what is transmitted); on a paged
# pool that is: pack the request's blocks, transfer, unpack into the receiver's free blocks.  These
# three are exact by definition (16-bit words copied verbatim), written with numpy indexing.

def _block_view(cache: np.ndarray, strides, num_kv_heads, block_size, head_dim) -> np.ndarray:
    """[NB, Hkv, bs, D] strided view of a uint16 pool addressed by (block, head, token) strides."""
    assert cache.dtype == np.uint16 and cache.flags.c_contiguous
    bstr, hstr, tstr = (int(s) for s in strides)
    nb = cache.size // bstr
    return np.lib.stride_tricks.as_strided(
        cache.reshape(-1), shape=(nb, num_kv_heads, block_size, head_dim),
        strides=(2 * bstr, 2 * hstr, 2 * tstr, 2), writeable=cache.flags.writeable)


def _valid(ids, nb):
    ids = np.asarray(ids, dtype=np.int64)
    return ids, (ids >= 0) & (ids < nb)


def gather_blocks(k_cache, v_cache, block_ids, *, num_kv_heads, block_size, head_dim, strides,
                  k_packed=None, v_packed=None):
    """Packed copies [n, Hkv, bs, D] of the listed pool blocks, in list order.  An id outside the
    pool leaves its packed block as it was (zeros when the buffers are created here)."""
    kv, vv = (_block_view(c, strides, num_kv_heads, block_size, head_dim) for c in (k_cache, v_cache))
    ids, ok = _valid(block_ids, kv.shape[0])
    shape = (ids.size, num_kv_heads, block_size, head_dim)
    k_packed = np.zeros(shape, np.uint16) if k_packed is None else k_packed
    v_packed = np.zeros(shape, np.uint16) if v_packed is None else v_packed
    k_packed[ok] = kv[ids[ok]]
    v_packed[ok] = vv[ids[ok]]
    return k_packed, v_packed


def scatter_blocks(k_packed, v_packed, block_ids, k_cache, v_cache, *, num_kv_heads, block_size, head_dim,
                   strides) -> None:
    """In place: pool block block_ids[i] <- packed block i (ids outside the pool are skipped)."""
    kv, vv = (_block_view(c, strides, num_kv_heads, block_size, head_dim) for c in (k_cache, v_cache))
    ids, ok = _valid(block_ids, kv.shape[0])
    kv[ids[ok]] = np.asarray(k_packed).reshape(ids.size, num_kv_heads, block_size, head_dim)[ok]
    vv[ids[ok]] = np.asarray(v_packed).reshape(ids.size, num_kv_heads, block_size, head_dim)[ok]


def copy_blocks(k_cache, v_cache, src_ids, dst_ids, *, num_kv_heads, block_size, head_dim, strides) -> None:
    """In place: pool block dst_ids[i] <- pool block src_ids[i]; every source is read before any
    destination is written (sources and destinations are disjoint by contract)."""
    kv, vv = (_block_view(c, strides, num_kv_heads, block_size, head_dim) for c in (k_cache, v_cache))
    src, oks = _valid(src_ids, kv.shape[0])
    dst, okd = _valid(dst_ids, kv.shape[0])
    ok = oks & okd
    ksrc, vsrc = kv[src[ok]].copy(), vv[src[ok]].copy()
    kv[dst[ok]] = ksrc
    vv[dst[ok]] = vsrc
