"""Pins of the 8-bit (E4M3) oracle: the format against an independent library conversion and
hand-worked cases; the attention against the bf16 oracle on the dequantised pool."""
import numpy as np
import pytest
import torch

import oracle


def test_decode_all_codes_against_library_and_definition():
    codes = np.arange(256, dtype=np.uint8)
    got = oracle.e4m3_decode(codes)
    lib = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(got), np.isnan(lib)) and np.isnan(got).sum() == 2          # 0x7F and 0xFF
    ok = ~np.isnan(got)
    assert np.array_equal(got[ok], lib[ok])
    # hand-worked: 0x38 = 0 0111 000 = 1.0; 0x7E = 448; 0x01 = 2^-9; 0x08 = 2^-6; 0xC4 = -(2^1 * 1.5) = -3
    assert got[0x38] == 1.0 and got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6
    assert got[0xC4] == -3.0 and got[0x00] == 0.0 and np.signbit(got[0x80])


def test_encode_ties_saturation_and_library():
    enc = lambda *xs: oracle.e4m3_encode(np.array(xs, dtype=np.float32)).tolist()
    # midpoints: 1.0 (0x38) | 1.125 (0x39) | 1.25 (0x3A): ties go to the even code
    assert enc(1.0625, 1.1875, 1.06251, 1.0624) == [0x38, 0x3A, 0x39, 0x38]
    assert enc(448.0, 449.0, 1e9, np.inf, -1e9, -np.inf, 464.0) == [0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0xFE, 0x7E]
    assert enc(0.0, -0.0, 2.0 ** -10, 2.0 ** -10 * 1.01, -(2.0 ** -11)) == [0x00, 0x80, 0x00, 0x01, 0x80]
    assert enc(np.nan) == [0x7F]
    # every code maps back to itself
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    assert np.array_equal(oracle.e4m3_encode(oracle.e4m3_decode(codes).astype(np.float32)), codes)
    # in range, the library's round-to-nearest-even conversion agrees
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4000) * s for s in (0.01, 1.0, 60.0)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(oracle.e4m3_encode(x), lib)


def _bf16_bits(x32: np.ndarray) -> np.ndarray:
    return torch.from_numpy(x32.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_attention_equals_bf16_oracle_on_the_dequantised_pool():
    rng = np.random.default_rng(1)
    B, Hq, Hkv, D, bs, NB = 3, 4, 2, 16, 4, 11
    lens = np.array([9, 1, 14], dtype=np.int32)
    table = np.stack([rng.permutation(NB)[:4] for _ in range(B)]).astype(np.int32)
    k8 = rng.integers(0, 256, (NB, Hkv, bs, D), dtype=np.uint8)
    v8 = rng.integers(0, 256, (NB, Hkv, bs, D), dtype=np.uint8)
    k8[(k8 & 0x7F) == 0x7F] = 0x10                       # no NaN codes
    v8[(v8 & 0x7F) == 0x7F] = 0x90
    q = _bf16_bits(rng.standard_normal((B, Hq, D)))
    ks, vs = 0.25, 2.0                                    # powers of two: dequantised values are exact in bf16
    strides = (Hkv * bs * D, bs * D, D)
    r8 = oracle.decode_attention_fp8(q, k8, v8, table, lens, 0.3, ks, vs, num_kv_heads=Hkv, block_size=bs, strides=strides)
    k16 = _bf16_bits(oracle.e4m3_decode(k8) * ks)
    v16 = _bf16_bits(oracle.e4m3_decode(v8) * vs)
    r16 = oracle.decode_attention(q, k16, v16, table, lens, 0.3, num_kv_heads=Hkv, block_size=bs, strides=strides)
    assert np.array_equal(r8.out, r16.out) and np.array_equal(r8.lse, r16.lse)
    assert np.allclose(r8.wsum, 1.0, atol=1e-12)


def test_append_quantises_one_slot_and_touches_nothing_else():
    rng = np.random.default_rng(2)
    B, Hkv, D, bs, NB = 3, 2, 16, 4, 9
    k8 = rng.integers(0, 256, (NB, Hkv, bs, D), dtype=np.uint8)
    v8 = rng.integers(0, 256, (NB, Hkv, bs, D), dtype=np.uint8)
    table = np.array([[3, 5, -1], [0, 8, 2], [7, 1, 6]], dtype=np.int32)
    pos = np.array([5, 11, 99], dtype=np.int32)           # block 5 slot 1; block 2 slot 3; beyond the table: skipped
    kn32 = rng.standard_normal((B, Hkv, D)).astype(np.float32) * 3
    vn32 = rng.standard_normal((B, Hkv, D)).astype(np.float32) * 300    # saturates here and there
    kn, vn = _bf16_bits(kn32), _bf16_bits(vn32)
    ks, vs = np.float32(0.37), np.float32(0.9)
    k2, v2 = k8.copy(), v8.copy()
    n = oracle.kv_append_fp8(kn, vn, k2, v2, table, pos, ks, vs, block_size=bs, strides=(Hkv * bs * D, bs * D, D))
    assert n == 2
    kb = torch.from_numpy(kn.view(np.int16).copy()).view(torch.bfloat16).float().numpy()
    vb = torch.from_numpy(vn.view(np.int16).copy()).view(torch.bfloat16).float().numpy()
    want_k, want_v = k8.copy(), v8.copy()
    for b, (blk, slot) in enumerate([(5, 1), (2, 3)]):
        want_k[blk, :, slot, :] = oracle.e4m3_encode((kb[b] / ks).astype(np.float32))
        want_v[blk, :, slot, :] = oracle.e4m3_encode((vb[b] / vs).astype(np.float32))
    assert np.array_equal(k2, want_k) and np.array_equal(v2, want_v)
    assert (want_v == 0x7E).any() or (want_v == 0xFE).any()
