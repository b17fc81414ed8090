"""8-bit (E4M3) KV cache on the GPU vs the fp64 oracle over the same codes, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs
from util import assert_parity

pytestmark = pytest.mark.gpu
G = inputs.LengthGroup
C = inputs.DecodeConfig


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def fixed(*vals):
    return (G(len(vals), min(vals), max(vals), "fixed", tuple(vals)),)


CASES = [
    # every tail length around tile / stage / block boundaries, and an empty sequence
    C("fp8-edges", 32, 8, 128, 16, fixed(0, 1, 2, 15, 16, 17, 31, 33, 63, 64, 65, 100, 127, 129, 191, 193, 300), seed=61,
      pool_fill=0.7, shuffle_batch=False),
    C("fp8-g1", 4, 4, 128, 16, (G(6, 1, 400),), seed=62),
    C("fp8-g5-bs32", 40, 8, 128, 32, (G(6, 1, 700),), seed=63, pool_fill=0.8),
    C("fp8-g8-bs32", 64, 8, 128, 32, (G(5, 1, 900),), seed=64, sigma=0.5),
    C("fp8-g16", 32, 2, 128, 16, (G(4, 1, 500),), seed=65),
    C("fp8-bs128", 16, 4, 128, 128, (G(5, 1, 900),), seed=66),
    C("fp8-token-major", 32, 8, 128, 16, (G(6, 1, 500),), seed=67, layout="token_major", pool_fill=0.75),
    C("fp8-split", 32, 8, 128, 16, fixed(5000, 37, 2049, 1025, 300, 9999), seed=68, pool_fill=0.9, shuffle_batch=False),
    C("fp8-split-g8-bs32", 64, 8, 128, 32, fixed(20000, 129, 4097, 64), seed=69, sigma=0.5, shuffle_batch=False),
]
K_SCALE, V_SCALE = 1.0 / 32, 0.04


def oracle8(batch, lens, k8, v8):
    cfg = batch.cfg
    return oracle.decode_attention_fp8(inputs.as_u16(batch.q), k8, v8, batch.block_table.cpu().numpy(),
                                       lens.cpu().numpy(), cfg.scale, K_SCALE, V_SCALE,
                                       num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size, strides=batch.strides)


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_attention_fp8_matches_oracle(cfg):
    b16 = inputs.make_batch(cfg, "cuda", poison=True, table_pad=2**31 - 1)
    batch = inputs.to_e4m3_pool(b16, K_SCALE, V_SCALE)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    out = torch.full_like(batch.q, float("nan"))
    binding.decode_attention_fp8(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                                 cfg.scale, K_SCALE, V_SCALE, out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle8(batch, batch.context_lens, inputs.as_u8(batch.k_cache), inputs.as_u8(batch.v_cache))
    assert_parity(out, ref.out, what=cfg.name)
    out2 = torch.full_like(out, float("nan"))
    binding.decode_attention_fp8(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                                 cfg.scale, K_SCALE, V_SCALE, out2, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))          # run-to-run bitwise


def test_single_token_returns_the_dequantised_value_row():
    cfg = C("fp8-t1", 8, 2, 128, 16, fixed(1, 1, 1), seed=70, shuffle_batch=False)
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=True), K_SCALE, V_SCALE)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(batch.q)
    binding.decode_attention_fp8(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                                 cfg.scale, K_SCALE, V_SCALE, out, ws)
    torch.cuda.synchronize()
    v8 = inputs.as_u8(batch.v_cache)
    table = batch.block_table.cpu().numpy()
    for b in range(3):
        for hq in range(8):
            want = oracle.e4m3_decode(v8[table[b, 0], hq // 4, 0, :]) * np.float32(V_SCALE)
            want = torch.tensor(want, dtype=torch.float32).to(torch.bfloat16)   # weight is exactly 1
            assert torch.equal(out[b, hq].cpu().view(torch.int16), want.view(torch.int16))


@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_append_fp8_bit_exact_over_the_whole_pool(layout):
    cfg = C("fp8-append", 32, 8, 128, 16, (G(40, 1, 600),), seed=71, pool_fill=0.8, layout=layout)
    b16 = inputs.make_batch(cfg, "cuda", poison=True)
    # new rows with values that saturate, hit ties and vanish
    b16.k_new.mul_(30.0)
    b16.v_new[::2] = (b16.v_new[::2] * 1e-3)
    b16.k_new[0, 0, :8] = torch.tensor([1.0625, 1.1875, 448.0, 500.0, -1e4, 0.0, -0.0, 2.0 ** -10]) * K_SCALE
    batch = inputs.to_e4m3_pool(b16, K_SCALE, V_SCALE)
    sh = binding.shape_of(batch)
    k_ref, v_ref = inputs.as_u8(batch.k_cache).copy(), inputs.as_u8(batch.v_cache).copy()
    n = oracle.kv_append_fp8(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k_ref, v_ref,
                             batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), K_SCALE, V_SCALE,
                             block_size=16, strides=batch.strides)
    assert n == cfg.batch
    binding.kv_append_fp8(sh, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                          batch.context_lens, K_SCALE, V_SCALE)
    torch.cuda.synchronize()
    assert np.array_equal(inputs.as_u8(batch.k_cache), k_ref) and np.array_equal(inputs.as_u8(batch.v_cache), v_ref)


def test_fused_step_fp8():
    cfg = C("fp8-step", 40, 8, 128, 16, (G(21, 1, 3000),), seed=72, pool_fill=0.85)
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=True), K_SCALE, V_SCALE)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    out = torch.full_like(batch.q, float("nan"))
    lens1 = (batch.context_lens + 1).contiguous()
    k_ref, v_ref = inputs.as_u8(batch.k_cache).copy(), inputs.as_u8(batch.v_cache).copy()
    binding.decode_step_fp8(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                            batch.context_lens, lens1, cfg.scale, K_SCALE, V_SCALE, out, ws)
    assert binding.workspace_status(ws) == 0
    oracle.kv_append_fp8(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k_ref, v_ref,
                         batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), K_SCALE, V_SCALE,
                         block_size=16, strides=batch.strides)
    assert np.array_equal(inputs.as_u8(batch.k_cache), k_ref) and np.array_equal(inputs.as_u8(batch.v_cache), v_ref)
    ref = oracle8(batch, lens1, k_ref, v_ref)
    assert_parity(out, ref.out, what="fp8 step")


def test_fp8_argument_errors():
    cfg = C("fp8-d64", 8, 2, 64, 16, fixed(5), seed=73)
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=False), 1.0, 1.0)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(batch.q)
    with pytest.raises(binding.OocoError) as e:
        binding.decode_attention_fp8(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                                     1.0, 1.0, 1.0, out, ws)
    assert e.value.status == -3                                               # head_dim 64 is not built
    cfg = C("fp8-scale", 8, 2, 128, 16, fixed(5), seed=74)
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=False), 1.0, 1.0)
    sh = binding.shape_of(batch)
    with pytest.raises(binding.OocoError) as e:
        binding.kv_append_fp8(sh, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                              batch.context_lens, 0.0, 1.0)
    assert e.value.status == -2
