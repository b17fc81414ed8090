"""Host-only checks of the C ABI: exported symbols, the byte/FLOP model, argument validation."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, fn)).read(), flags=re.S)
            names |= set(re.findall(r"\b(ooco_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert len(names) >= 10
    L = binding.lib()
    for n in names:
        assert hasattr(L, n), n
    from paper_2511_21862_b200 import sched
    assert set(names) == set(binding.EXPORTS) | set(sched.SCHED_EXPORTS)
    assert L.ooco_version() == 1
    assert binding.status_string(0) == "ok" and "unknown" in binding.status_string(-99)


def read_golden():
    rows = []
    for line in open(os.path.join(ROOT, "tests", "golden", "bytes_model.txt")):
        if line.startswith("#") or not line.strip():
            continue
        a, b, c = (p.split() for p in line.split("|"))
        rows.append(([int(x) for x in a], [int(x) for x in b], [int(x) for x in c]))
    return rows


@pytest.mark.parametrize("row", read_golden(), ids=lambda r: "-".join(map(str, r[0])))
def test_bytes_model_golden(row):
    (Hq, Hkv, D, bs, d), lens, want = row
    keys = oracle.COST_FIELDS
    got_o = oracle.bytes_model(lens, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, block_size=bs, bytes_per_value=d)
    assert [got_o[k] for k in keys] == want
    sh = binding.Shape(len(lens), Hq, Hkv, D, bs, 1, 1, Hkv * bs * D, bs * D, D)
    got_l = binding.decode_bytes_model(sh, torch.tensor(lens, dtype=torch.int32), d)
    assert [got_l[k] for k in keys] == want


def test_bytes_model_equals_enumeration_of_addressed_slots():
    """bytes_kv = bytes of the distinct cache words a batch addresses; index = table + length words."""
    cfg = inputs.DecodeConfig("enum", 12, 3, 64, 16, (inputs.LengthGroup(5, 1, 90),), seed=21, pool_fill=0.6)
    batch = inputs.make_batch(cfg)
    lens = batch.context_lens
    touched = set()
    table_words = 0
    for b in range(5):
        T = int(lens[b])
        table_words += -(-T // 16)
        for t in range(T):
            blk = int(batch.block_table[b, t // 16])
            for h in range(3):
                touched.add((blk, h, t % 16))
    kv_bytes = 2 * len(touched) * 64 * 2                      # K and V, D elements of 2 bytes
    o = oracle.bytes_model(lens.numpy(), num_q_heads=12, num_kv_heads=3, head_dim=64, block_size=16)
    l = binding.decode_bytes_model(binding.shape_of(batch), lens.contiguous())
    for got in (o, l):
        assert got["bytes_kv"] == kv_bytes
        assert got["bytes_index"] == 4 * (5 + table_words)
        assert got["bytes_q"] == got["bytes_out"] == batch.q.numel() * 2
        assert got["flops"] == 2 * 2 * 12 * 64 * int(lens.sum())   # QK^T and PV, 2 flops per MAC
        assert got["bytes_paper"] == got["bytes_q"] + got["bytes_out"] + got["bytes_kv"]


def test_bytes_model_mha_matches_printed_table_entry():
    """With Hq == Hkv the table's printed ratio is 1: memory = 2d(Sq*Dh + Skv*Dh)."""
    lens = torch.tensor([7, 300, 4096], dtype=torch.int32)
    Hq, D, d = 16, 128, 2
    sh = binding.Shape(3, Hq, Hq, D, 16, 1, 1, Hq * 16 * D, 16 * D, D)
    got = binding.decode_bytes_model(sh, lens, d)
    Dh = Hq * D
    assert got["bytes_paper"] == sum(2 * d * (1 * Dh + int(t) * Dh) for t in lens)
    assert got["flops"] == sum(4 * Dh * 1 * int(t) for t in lens)


def test_argument_validation_without_a_device():
    L = binding.lib()
    good = binding.Shape(2, 8, 2, 64, 16, 8, 4, 2 * 16 * 64, 16 * 64, 64)
    assert binding.workspace_bytes(good) > 256 and binding.step_staging_bytes(good) > 0
    one = ctypes.c_void_p(256)
    def attn(shape, ptr=one, ws_bytes=1 << 40):
        return L.ooco_decode_attention(ctypes.byref(shape.c()), ptr, ptr, ptr, ptr, ptr, 1.0, ptr, ptr, ws_bytes, None)
    import dataclasses
    assert attn(good, ptr=None) == -1                                                   # NULLPTR
    assert attn(dataclasses.replace(good, num_q_heads=7)) == -2                         # Hq % Hkv
    assert attn(dataclasses.replace(good, batch=0)) == -2
    assert attn(dataclasses.replace(good, head_dim=96, kv_token_stride=96)) == -3       # UNSUPPORTED
    assert attn(dataclasses.replace(good, block_size=8)) == -3
    assert attn(dataclasses.replace(good, num_q_heads=64, num_kv_heads=2)) == -3        # group of 32
    assert attn(dataclasses.replace(good, kv_token_stride=68)) == -3                    # not 16-byte multiple
    assert attn(good, ws_bytes=1024) == -4                                              # WORKSPACE
    # the softmax scale must be positive and finite (every kernel may then take the maximum before scaling)
    for bad_scale in (0.0, -0.125, float("inf"), float("nan")):
        assert L.ooco_decode_attention(ctypes.byref(good.c()), one, one, one, one, one, bad_scale, one, one, 1 << 40,
                                       None) == -2
        assert L.ooco_decode_step_host(ctypes.byref(good.c()), one, one, one, one, one, one, one, one, bad_scale, one,
                                       one, 1 << 40, one, 1 << 40, None) == -2
    # the host-buffer step checks both scratch buffers before it enqueues its first copy
    assert L.ooco_decode_step_host(ctypes.byref(good.c()), one, one, one, one, one, one, one, one, 1.0, one,
                                   one, 1 << 40, one, 1024, None) == -4
    assert L.ooco_kv_append(ctypes.byref(good.c()), None, one, one, one, one, one, None) == -1
    assert L.ooco_decode_bytes_model(ctypes.byref(good.c()), None, 2, None) == -1
    assert L.ooco_set_tuning(99, 1) == -2 and L.ooco_set_tuning(0, 3) == -2
    bad = dataclasses.replace(good, head_dim=96, kv_token_stride=96)
    assert L.ooco_decode_workspace_bytes(ctypes.byref(bad.c())) == 0


def test_query_length_limits_and_workspace_growth_without_a_device():
    """Host-side rules of the several-query-token entry points: q_len in [1, 8192]; the workspace holds one
    fp32 partial row per (split item, score column), so it grows with q_len within a kernel family; q_len = 1 is
    the decode size;
    a misaligned q or out pointer is refused before anything is launched."""
    L = binding.lib()
    sh = binding.Shape(4, 32, 8, 128, 16, 1000, 64, 8 * 16 * 128, 16 * 128, 128)
    assert binding.workspace_bytes_mq(sh, 1) == binding.workspace_bytes(sh)
    for qs in ((1, 2, 4), (5, 16, 64, 1024, 8192)):      # decode kernels / prefill-chunk kernels (they plan fewer items)
        sizes = [binding.workspace_bytes_mq(sh, q) for q in qs]
        assert all(a < b for a, b in zip(sizes, sizes[1:]))
    for q in (0, -1, 8193):
        with pytest.raises(binding.OocoError):
            binding.workspace_bytes_mq(sh, q)
    ok, odd = ctypes.c_void_p(256), ctypes.c_void_p(258)
    def attn(q_len, q=ok, out=ok, ws_bytes=1 << 40):
        return L.ooco_decode_attention_mq(ctypes.byref(sh.c()), q_len, q, ok, ok, ok, ok, 1.0, out, ok, ws_bytes, None)
    assert attn(8193) == -3 and attn(0) == -2
    assert attn(64, q=odd) == -3 and attn(64, out=odd) == -3
    assert attn(64, ws_bytes=binding.workspace_bytes_mq(sh, 4)) == -4
    assert L.ooco_set_tuning(11, 0) == 0 and L.ooco_set_tuning(11, 1) == 0 and L.ooco_set_tuning(12, 1) == 0 and L.ooco_set_tuning(16, 1) == -2
    assert L.ooco_set_tuning(15, 0) == 0 and L.ooco_set_tuning(15, 3) == -2 and L.ooco_set_tuning(15, 1) == 0   # two-tile chunk kernel
    assert L.ooco_set_tuning(15, 2) == 0
    # knob 12: off, every prefill chunk, or a first column count of 17 or more
    assert L.ooco_set_tuning(12, 16) == -2 and L.ooco_set_tuning(12, 33) == 0 and L.ooco_set_tuning(12, 0) == 0
    assert L.ooco_set_tuning(12, 1) == 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libooco.so")
    with pytest.raises(ImportError):
        binding.lib()


def test_block_movement_and_fp8_argument_validation_needs_no_device():
    """Bad arguments are refused on the host before any CUDA call (this runs without a GPU)."""
    L = binding.lib()
    sh = binding.Shape(1, 8, 8, 128, 16, 10, 1, 8 * 16 * 128, 16 * 128, 128).c()
    p = ctypes.c_void_p
    buf = (ctypes.c_uint8 * 64)()
    a = ctypes.addressof(buf)
    a16 = (a + 15) & ~15
    assert L.ooco_kv_gather_blocks(ctypes.byref(sh), None, p(a16), p(a16), 1, p(a16), p(a16), None, None) == -1
    assert L.ooco_kv_gather_blocks(ctypes.byref(sh), p(a16), p(a16), p(a16), -1, p(a16), p(a16), None, None) == -2
    assert L.ooco_kv_scatter_blocks(ctypes.byref(sh), p(a16 + 2), p(a16), p(a16), 1, p(a16), p(a16), None, None) == -3
    assert L.ooco_kv_copy_blocks(ctypes.byref(sh), p(a16), p(a16), None, p(a16), 1, None, None) == -1
    assert L.ooco_kv_gather_blocks(ctypes.byref(sh), p(a16), p(a16), None, 0, p(a16), p(a16), None, None) == 0   # n = 0
    bad = binding.Shape(1, 8, 8, 64, 16, 10, 1, 8 * 16 * 64, 16 * 64, 64).c()
    f = ctypes.c_float
    assert L.ooco_kv_append_fp8(ctypes.byref(bad), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), f(1), f(1), None) == -3
    assert L.ooco_kv_append_fp8(ctypes.byref(sh), p(a16), p(a16), p(a16), p(a16), p(a16), p(a16), f(-1), f(1), None) == -2
    assert L.ooco_decode_attention_fp8(ctypes.byref(sh), p(a16), p(a16), p(a16), p(a16), p(a16), f(1), f(1), f(0),
                                       p(a16), p(a16), 0, None) == -2


def test_attention_bytes_model_with_several_query_tokens():
    """Against the scheduling oracle's literal table row, summed over the batch; q_len = 1 is the decode model."""
    from oracle import sched_oracle as so
    rng = np.random.default_rng(4)
    for Hq, Hkv, D, d, Sq in [(32, 8, 128, 2, 1), (32, 8, 128, 2, 4), (40, 8, 128, 1, 3), (8, 8, 64, 2, 16)]:
        lens = rng.integers(0, 9000, 23).astype(np.int32)
        sh = binding.Shape(len(lens), Hq, Hkv, D, 16, 1, 1, Hkv * 16 * D, 16 * D, D)
        got = binding.attention_bytes_model(sh, Sq, torch.from_numpy(lens), d)
        fl = by = 0
        for T in lens:
            f, b = so.attention_cost(Hq * D, Sq, int(T), Hq, Hkv, d)
            fl, by = fl + f, by + b
        assert (got["flops"], got["bytes_paper"]) == (fl, by)
        assert got["bytes_q"] == got["bytes_out"] == d * Sq * Hq * D * len(lens)
        if Sq == 1:
            assert got == binding.decode_bytes_model(sh, torch.from_numpy(lens), d)


def test_range_predicates_of_the_checked_build():
    """The predicates the checked build guards its accesses with, evaluated on the host: each accepts the
    whole legal range and refuses the first value on either side of it."""
    P = binding.check_predicate
    NB = 1000
    assert P(0, 0, NB) and P(0, NB - 1, NB)
    assert not P(0, -1, NB) and not P(0, NB, NB) and not P(0, 2**31 - 1, NB) and not P(0, -7, NB)
    assert P(1, 0, 5) and P(1, 4, 5) and not P(1, 5, 5) and not P(1, -1, 5) and not P(1, 0, 0)
    # work item {sequence, slot, t0, t1, B, max_items, capacity in tokens}
    ok = (3, 17, 64, 128, 4, 18, 128)
    assert P(2, *ok)
    assert P(2, 0, 0, 0, 0, 4, 18, 128)                                            # an empty chunk at the start is in range
    for i, bad in ((0, -1), (0, 4), (1, -1), (1, 18), (2, -64), (2, 192), (3, 63), (3, 129)):
        args = list(ok)
        args[i] = bad
        assert not P(2, *args), (i, bad)
    # span {offset, bytes, lo, hi}: [offset, offset + bytes) inside [lo, hi)
    assert P(3, 1024, 4096, 1024, 5120) and P(3, 1024, 0, 1024, 1024)
    assert not P(3, 1023, 16, 1024, 5120) and not P(3, 5105, 16, 1024, 5120) and not P(3, 2048, -16, 1024, 5120)
    with pytest.raises(binding.OocoError):
        P(9, 0, 0)
    assert binding.checked_build() is False


def test_fp32_output_knob_is_a_switch():
    assert binding.get_tuning("out_f32") == 0
    L = binding.lib()
    assert L.ooco_set_tuning(13, 2) == -2 and L.ooco_set_tuning(16, 1) == -2 and L.ooco_get_tuning(99) == -2
    binding.set_tuning(out_f32=1)
    try:
        assert binding.get_tuning("out_f32") == 1
        good = binding.Shape(2, 8, 2, 64, 16, 8, 4, 2 * 16 * 64, 16 * 64, 64)
        one = ctypes.c_void_p(256)
        # the host-buffer step has no fp32 result buffer: refused before anything is enqueued
        assert L.ooco_decode_step_host(ctypes.byref(good.c()), one, one, one, one, one, one, one, one, 1.0, one,
                                       one, 1 << 40, one, 1 << 40, None) == -3
    finally:
        binding.set_tuning(out_f32=0)
