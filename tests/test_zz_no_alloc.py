"""ooco_decode_attention_static: the decode attention for callers that cannot allocate device memory.

Some users of this library have no way to call cudaMalloc when a decode step runs: the serving
engine gave the whole device to its KV pool at start-up, or the decode loop cannot afford the
device-wide synchronisation an allocation implies, or the host framework forbids allocations outside
its own pool.  For them the library carries a 16 MiB scratch array in its device image and an entry
point that uses it instead of a caller-provided workspace.  These tests call that entry point through
the C ABI, several times in a row on different batches (the shared array still holds the previous
call's contents), and require its output to be bit for bit the ordinary entry point's (both run the same
launches on the same plan), to match the fp64 oracle within the parity tolerance, and the call to
leave the device's free memory and torch's allocation counter untouched.

This file is collected last on purpose: a failure here cannot hide another test's result in a run
that stops at the first failure.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs

MAX_ABS_TOL, MEAN_ABS_TOL = 1e-2, 1e-3          # the tolerance of the parity tests
G, C = inputs.LengthGroup, inputs.DecodeConfig


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def both_entry_points(cfg):
    batch = inputs.make_batch(cfg, "cuda", poison=True, table_pad=-1)
    sh = binding.shape_of(batch)
    assert binding.workspace_bytes(sh) <= binding.STATIC_SCRATCH_BYTES
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    want = torch.full_like(batch.q, float("nan"))
    got = torch.full_like(batch.q, float("nan"))
    binding.decode_attention(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                             cfg.scale, want, ws)
    assert binding.workspace_status(ws) == 0
    binding.decode_attention_static(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table,
                                    batch.context_lens, cfg.scale, got)
    torch.cuda.synchronize()
    return batch, got, want


@pytest.mark.gpu
def test_static_scratch_entry_point_matches_the_workspace_one_twice_in_a_row():
    first = C("noalloc-a", 32, 8, 128, 16, (G(20, 1, 2500), G(2, 5000, 7000)), seed=60, pool_fill=0.8)   # split + unsplit
    second = C("noalloc-b", 8, 2, 64, 32, (G(7, 0, 300),), seed=61)                                        # other shape, stale scratch
    for cfg in (first, second, first):
        batch, got, want = both_entry_points(cfg)
        assert not torch.isnan(got.float()).any()
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), cfg.name       # same launches, same plan
        ref = oracle.decode_attention(inputs.as_u16(batch.q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
                                      batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                      num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size, strides=batch.strides)
        err = np.abs(got.double().cpu().numpy() - ref.out)
        assert err.max() <= MAX_ABS_TOL and err.mean() <= MEAN_ABS_TOL, (cfg.name, err.max(), err.mean())


@pytest.mark.gpu
def test_static_scratch_entry_point_allocates_nothing_after_its_first_call():
    """After one warm-up call on the device (module loading and the symbol look-up happen there) a call
    changes neither the device's free memory nor the bytes torch has handed out."""
    cfg = C("noalloc-c", 32, 8, 128, 16, (G(12, 1, 3000),), seed=62)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    out = torch.empty_like(batch.q)
    call = lambda: binding.decode_attention_static(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table,
                                                   batch.context_lens, cfg.scale, out)
    call()
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (held0, reserved0)


def test_static_scratch_entry_point_rejects_shapes_beyond_its_array():
    """Host-side check only (nothing is launched): a cfg4-sized batch needs more than 16 MiB."""
    big = binding.Shape(512, 32, 8, 128, 16, 1000, 1025, 8 * 16 * 128, 16 * 128, 128)
    assert binding.workspace_bytes(big) > binding.STATIC_SCRATCH_BYTES
    one = ctypes.c_void_p(256)
    rc = binding.lib().ooco_decode_attention_static(ctypes.byref(big.c()), one, one, one, one, one, 1.0, one, None)
    assert rc == -4
    detail = binding.lib().ooco_last_error_detail().decode()
    assert "built-in scratch" in detail and str(binding.STATIC_SCRATCH_BYTES) in detail
    bad = binding.Shape(0, 32, 8, 128, 16, 1000, 1025, 8 * 16 * 128, 16 * 128, 128)
    assert binding.lib().ooco_decode_attention_static(ctypes.byref(bad.c()), one, one, one, one, one, 1.0, one, None) == -2
