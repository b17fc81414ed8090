"""Several query tokens per sequence (S_q > 1) on the GPU vs the oracle, through the C ABI."""
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


def run_case(cfg, Sq, seed):
    batch = inputs.make_batch(cfg, "cuda", poison=True, table_pad=2**31 - 1)
    B, Hq, D = cfg.batch, cfg.num_q_heads, cfg.head_dim
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = (torch.randn((B, Sq, Hq, D), generator=g, device="cuda") * cfg.sigma).to(torch.bfloat16)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_attention_mq(sh, q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                                cfg.scale, out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle.decode_attention_mq(inputs.as_u16(q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
                                     batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                     num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size, strides=batch.strides)
    assert_parity(out.reshape(B * Sq, Hq, D), ref.out.reshape(B * Sq, Hq, D), what=f"{cfg.name} Sq={Sq}")
    return batch, q, out, ref


CASES = [
    # lengths around tile / stage / block boundaries; some contexts hold nothing but (part of) the queries
    (C("mq-edges-g4", 32, 8, 128, 16, fixed(0, 1, 2, 3, 4, 15, 16, 17, 18, 19, 63, 64, 65, 66, 67, 127, 128, 129, 130, 300),
       seed=81, pool_fill=0.7, shuffle_batch=False), 4),
    (C("mq-g4-sq2", 32, 8, 128, 16, (G(8, 1, 600),), seed=82), 2),
    (C("mq-g1-sq16", 8, 8, 128, 16, (G(6, 1, 500),), seed=83), 16),
    (C("mq-g8-sq2-bs32", 64, 8, 128, 32, (G(5, 1, 900),), seed=84, sigma=0.5), 2),
    (C("mq-g5-sq3", 40, 8, 128, 32, (G(6, 1, 700),), seed=85), 3),
    (C("mq-d64-g4-sq3", 8, 2, 64, 16, (G(6, 1, 400),), seed=86), 3),
    (C("mq-token-major", 32, 8, 128, 16, (G(6, 1, 500),), seed=87, layout="token_major"), 4),
    # split into several chunks; chunk boundaries fall inside the last few tokens for some
    (C("mq-split", 32, 8, 128, 16, fixed(5000, 37, 2049, 2050, 2051, 1025, 300, 9999), seed=88, pool_fill=0.9,
       shuffle_batch=False), 4),
    (C("mq-split-g2-sq8", 16, 8, 128, 16, fixed(7000, 129, 4097, 4100, 64), seed=89, shuffle_batch=False), 8),
]


@pytest.mark.parametrize("cfg,Sq", CASES, ids=lambda v: getattr(v, "name", str(v)))
def test_multi_query_matches_oracle(cfg, Sq):
    run_case(cfg, Sq, seed=cfg.seed)


# More than 16 score columns per (sequence, kv head): the prefill-chunk kernel (row tiles of 32 / 64 / 128
# columns).  Contexts shorter than, equal to and just above the chunk; ragged last row tile; every block size.
CHUNK_CASES = [
    # 20 columns.  (sigma 0.5: with contexts of a few tokens the rows are single V entries or means of a few, and at
    # |out| >= 2 the rounding of the bf16 output, 2^-7, plus that of the bf16 weights, 2^-9 |v|, alone passes 1e-2)
    (C("ck-g4-sq5", 32, 8, 128, 16, fixed(0, 1, 4, 5, 6, 63, 64, 65, 129, 700), seed=101, pool_fill=0.7,
       shuffle_batch=False, sigma=0.5), 5),
    (C("ck-g4-sq16", 32, 8, 128, 16, fixed(3, 16, 17, 64, 100, 1000), seed=102, shuffle_batch=False), 16),   # 64 columns
    (C("ck-g4-sq33", 32, 8, 128, 16, fixed(33, 34, 200, 1500), seed=103, shuffle_batch=False), 33),          # 132: ragged tile
    (C("ck-g4-sq128-fresh", 32, 8, 128, 16, fixed(128, 128, 500, 1290), seed=104, shuffle_batch=False), 128),  # T = S_q: a whole prompt
    (C("ck-g5-sq7-bs32", 40, 8, 128, 32, (G(5, 7, 900),), seed=105), 7),
    (C("ck-g8-sq64-bs64", 64, 8, 128, 64, (G(3, 64, 1200),), seed=106, sigma=0.5), 64),
    (C("ck-g1-sq100-bs128", 8, 8, 128, 128, (G(4, 100, 800),), seed=107), 100),
    (C("ck-d64-g4-sq40", 8, 2, 64, 16, (G(6, 1, 900),), seed=108), 40),
    (C("ck-token-major", 32, 8, 128, 16, (G(4, 50, 600),), seed=109, layout="token_major"), 24),
    # split into several chunks (few long sequences)
    (C("ck-split", 32, 8, 128, 16, fixed(9000, 2049, 70), seed=110, pool_fill=0.9, shuffle_batch=False), 48),
    (C("ck-split-g2", 16, 8, 128, 16, fixed(20000, 4100), seed=111, shuffle_batch=False), 9),
    # 320 columns: a pair of 128-row tiles, then a pair whose second tile has no rows; contexts around the slot size
    # (sigma 0.5: the first queries of a fresh prompt return single V entries, whose bf16 rounding alone would pass
    # 1e-2 beyond |v| = 2.56)
    (C("ck-g4-sq80", 32, 8, 128, 16, fixed(80, 81, 127, 128, 129, 208, 2600, 9100), seed=112, pool_fill=0.8,
       shuffle_batch=False, sigma=0.5), 80),
    # up to 128 columns on the kernel's one-tile mode: many short units (one to four 128-token slots each, contexts
    # shorter than the chunk included), so that unit boundaries, stages without tokens and the end marker come close
    # together; then exactly 128 columns with blocks of 32 tokens
    (C("ck-g4-sq10-short", 32, 8, 128, 16, (G(48, 1, 400),), seed=113, pool_fill=0.8), 10),
    (C("ck-g8-sq16-bs32", 64, 8, 128, 32, (G(24, 16, 700),), seed=114, sigma=0.5), 16),
]


@pytest.mark.parametrize("cfg,Sq", CHUNK_CASES, ids=lambda v: getattr(v, "name", str(v)))
def test_prefill_chunk_matches_oracle(cfg, Sq):
    run_case(cfg, Sq, seed=cfg.seed)


@pytest.mark.parametrize("cfg,Sq", [c for c in CHUNK_CASES if c[0].name in
                                    ("ck-g4-sq5", "ck-g4-sq33", "ck-g4-sq128-fresh", "ck-g8-sq64-bs64", "ck-split",
                                     "ck-split-g2", "ck-token-major")],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_prefill_chunk_on_the_mma_sync_kernel(cfg, Sq):
    """Prefill chunks at head_dim 128 run the tcgen05 kernels by default; the mma.sync kernel of the same
    shape stays selectable and must agree with the oracle too."""
    binding.set_tuning(chunk_tcgen05=0)
    try:
        run_case(cfg, Sq, seed=cfg.seed)
    finally:
        binding.set_tuning(chunk_tcgen05=1)


@pytest.mark.parametrize("two_tiles", [0, 1], ids=["never-two-tiles", "two-tiles-beyond-128-columns"])
@pytest.mark.parametrize("cfg,Sq", [c for c in CHUNK_CASES if c[0].name in
                                    ("ck-g4-sq5", "ck-g4-sq16", "ck-g4-sq33", "ck-g4-sq128-fresh", "ck-g8-sq64-bs64",
                                     "ck-split", "ck-g4-sq80", "ck-g4-sq10-short")],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_prefill_chunk_on_the_one_tile_tcgen05_kernel(cfg, Sq, two_tiles):
    """Over a bf16 cache the kernel with one CTA per SM (two 128-row tiles, or one tile in its one-tile mode) runs
    every chunk by default; the kernel with one tile per CTA and two CTAs per SM stays selectable, for all chunks
    or for those of up to 128 columns, and must agree with the oracle too."""
    binding.set_tuning(chunk_two_tiles=two_tiles)
    try:
        run_case(cfg, Sq, seed=cfg.seed)
    finally:
        binding.set_tuning(chunk_two_tiles=2)


def test_chunk_rows_agree_with_decode_rows():
    """A chunk of 8 query tokens (32 columns: chunk kernel) and two calls of 4 (16 columns: decode kernel)
    over the same cache compute the same rows, up to the rounding of a different summation order."""
    cfg = C("ck-vs-mq", 32, 8, 128, 16, (G(6, 8, 900),), seed=112)
    batch, q, out, _ = run_case(cfg, 8, seed=2)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, 4), dtype=torch.uint8, device="cuda")
    q_hi = q[:, 4:].contiguous()
    out_hi = torch.empty_like(q_hi)
    binding.decode_attention_mq(sh, q_hi, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                                cfg.scale, out_hi, ws)
    torch.cuda.synchronize()
    assert float((out[:, 4:].float() - out_hi.float()).abs().max()) <= 4e-3


def test_last_query_token_equals_single_query_call():
    """The last query token sees the whole context: the same result as ooco_decode_attention on that
    token, up to the rounding of a different summation order (the launch shape depends on the number
    of score columns)."""
    cfg = C("mq-vs-single", 32, 8, 128, 16, (G(10, 3, 200),), seed=90)
    batch, q, out, _ = run_case(cfg, 3, seed=1)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    q1 = q[:, -1].contiguous()
    out1 = torch.empty_like(q1)
    binding.decode_attention(sh, q1, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens, cfg.scale,
                             out1, ws)
    torch.cuda.synchronize()
    assert float((out[:, -1].float() - out1.float()).abs().max()) <= 4e-3            # a bf16 ulp or two at |x| < 1


def test_append_mq_bit_exact_then_attend():
    cfg = C("mq-append", 32, 8, 128, 16, (G(20, 1, 700),), seed=91, pool_fill=0.8)
    Sq = 4
    # room for Sq new tokens: draw the batch with contexts Sq - 1 longer, then treat the tail as not yet written
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    lens = batch.context_lens
    short = torch.clamp(lens - (Sq - 1), min=0).contiguous()             # positions of the first new token
    ok = (lens >= Sq - 1)
    g = torch.Generator(device="cuda").manual_seed(5)
    k_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    v_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    positions = torch.where(ok, short, torch.full_like(short, -100)).contiguous()   # too-short sequences: skipped
    sh = binding.shape_of(batch)
    k_ref, v_ref = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    table = batch.block_table.cpu().numpy()
    for i in range(Sq):                                                    # oracle: one token at a time
        oracle.kv_append(inputs.as_u16(k_new[:, i].contiguous()), inputs.as_u16(v_new[:, i].contiguous()), k_ref, v_ref,
                         table, (positions + i).cpu().numpy() * ok.cpu().numpy() - 100 * (~ok).cpu().numpy(),
                         block_size=16, strides=batch.strides)
    binding.kv_append_mq(sh, k_new, v_new, batch.k_cache, batch.v_cache, batch.block_table, positions)
    torch.cuda.synchronize()
    assert np.array_equal(inputs.as_u16(batch.k_cache), k_ref) and np.array_equal(inputs.as_u16(batch.v_cache), v_ref)


def test_unsupported_shapes_are_refused():
    cfg = C("mq-too-wide", 64, 8, 128, 16, fixed(50), seed=92)
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=False), 1.0, 1.0)
    sh = binding.shape_of(batch)
    with pytest.raises(binding.OocoError):
        binding.workspace_bytes_mq(sh, 8193)                               # beyond the largest chunk
    # the 8-bit cache is built for head_dim 128 only (refused on the host, before anything is launched)
    import ctypes
    sh64 = binding.Shape(1, 8, 2, 64, 16, 8, 4, 2 * 16 * 64, 16 * 64, 64)
    one = ctypes.c_void_p(256)
    assert binding.lib().ooco_decode_step_mq_fp8(ctypes.byref(sh64.c()), 3, one, None, None, one, one, one, None, one,
                                                 1.0, 1.0, 1.0, one, one, 1 << 40, None) == -3
    # a workspace sized for fewer query tokens is refused
    b16 = inputs.make_batch(cfg, "cuda", poison=False)
    sh16 = binding.shape_of(b16)
    small = torch.empty(binding.workspace_bytes_mq(sh16, 2), dtype=torch.uint8, device="cuda")
    q = torch.zeros((1, 64, 64, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.OocoError):
        binding.decode_attention_mq(sh16, q, b16.k_cache, b16.v_cache, b16.block_table, b16.context_lens, 1.0,
                                    torch.empty_like(q), small)


def test_fused_step_mq():
    """ooco_decode_step_mq = append of q_len tokens (bit-exact over the whole pool) + causal attention."""
    cfg = C("mq-step", 32, 8, 128, 16, (G(14, 4, 2600),), seed=93, pool_fill=0.85)
    Sq = 4
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    g = torch.Generator(device="cuda").manual_seed(6)
    q = torch.randn((cfg.batch, Sq, 32, 128), generator=g, device="cuda").to(torch.bfloat16)
    k_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    v_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    lens = batch.context_lens                                              # contexts INCLUDING the new tokens
    positions = (lens - Sq).contiguous()
    k_ref, v_ref = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    table = batch.block_table.cpu().numpy()
    for i in range(Sq):
        oracle.kv_append(inputs.as_u16(k_new[:, i].contiguous()), inputs.as_u16(v_new[:, i].contiguous()), k_ref, v_ref,
                         table, (positions + i).cpu().numpy(), block_size=16, strides=batch.strides)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_step_mq(sh, q, k_new, v_new, batch.k_cache, batch.v_cache, batch.block_table, positions, lens,
                           cfg.scale, out, ws)
    assert binding.workspace_status(ws) == 0 and binding.last_launch_count() == 3
    assert np.array_equal(inputs.as_u16(batch.k_cache), k_ref) and np.array_equal(inputs.as_u16(batch.v_cache), v_ref)
    ref = oracle.decode_attention_mq(inputs.as_u16(q), k_ref, v_ref, table, lens.cpu().numpy(), cfg.scale,
                                     num_kv_heads=8, block_size=16, strides=batch.strides)
    assert_parity(out.reshape(-1, 32, 128), ref.out.reshape(-1, 32, 128), what="fused mq step")


@pytest.mark.parametrize("Sq,tc", [(5, 1), (5, 0), (40, 1), (40, 0)],
                         ids=["20-columns-tcgen05", "20-columns-mma-sync", "160-columns-tcgen05", "160-columns-mma-sync"])
def test_fused_step_prefill_chunk(Sq, tc):
    """ooco_decode_step_mq with a chunk long enough for the prefill-chunk kernels: the fused append of q_len
    tokens (bit-exact over the whole pool) is seen by the attention of the same call."""
    cfg = C("ck-step", 32, 8, 128, 16, (G(6, 40, 1500),), seed=120, pool_fill=0.85)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    g = torch.Generator(device="cuda").manual_seed(9)
    q = torch.randn((cfg.batch, Sq, 32, 128), generator=g, device="cuda").to(torch.bfloat16)
    k_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    v_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    lens = batch.context_lens                                              # contexts INCLUDING the new tokens
    positions = (lens - Sq).contiguous()
    k_ref, v_ref = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    table = batch.block_table.cpu().numpy()
    for i in range(Sq):
        oracle.kv_append(inputs.as_u16(k_new[:, i].contiguous()), inputs.as_u16(v_new[:, i].contiguous()), k_ref, v_ref,
                         table, (positions + i).cpu().numpy(), block_size=16, strides=batch.strides)
    binding.set_tuning(chunk_tcgen05=tc)
    try:
        ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
        out = torch.full_like(q, float("nan"))
        binding.decode_step_mq(sh, q, k_new, v_new, batch.k_cache, batch.v_cache, batch.block_table, positions, lens,
                               cfg.scale, out, ws)
        assert binding.workspace_status(ws) == 0 and binding.last_launch_count() == 3
    finally:
        binding.set_tuning(chunk_tcgen05=1)
    assert np.array_equal(inputs.as_u16(batch.k_cache), k_ref) and np.array_equal(inputs.as_u16(batch.v_cache), v_ref)
    ref = oracle.decode_attention_mq(inputs.as_u16(q), k_ref, v_ref, table, lens.cpu().numpy(), cfg.scale,
                                     num_kv_heads=8, block_size=16, strides=batch.strides)
    assert_parity(out.reshape(-1, 32, 128), ref.out.reshape(-1, 32, 128), what=f"fused chunk step Sq={Sq}")


@pytest.mark.parametrize("cfg,Sq", [
    (C("mq8-edges", 32, 8, 128, 16, fixed(0, 1, 2, 3, 4, 15, 16, 17, 18, 63, 64, 65, 66, 127, 129, 300), seed=94,
       pool_fill=0.7, shuffle_batch=False), 4),
    (C("mq8-g8-sq2", 64, 8, 128, 32, (G(5, 1, 900),), seed=95, sigma=0.5), 2),
    (C("mq8-split", 32, 8, 128, 16, fixed(5000, 37, 2049, 2050, 2051, 300), seed=96, shuffle_batch=False), 3),
], ids=lambda v: getattr(v, "name", str(v)))
def test_multi_query_over_8bit_cache(cfg, Sq):
    ks, vs = 1.0 / 32, 0.04
    b16 = inputs.make_batch(cfg, "cuda", poison=True, table_pad=2**31 - 1)
    batch = inputs.to_e4m3_pool(b16, ks, vs)
    B, Hq, D = cfg.batch, cfg.num_q_heads, cfg.head_dim
    g = torch.Generator(device="cuda").manual_seed(cfg.seed)
    q = (torch.randn((B, Sq, Hq, D), generator=g, device="cuda") * cfg.sigma).to(torch.bfloat16)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_step_mq_fp8(sh, q, None, None, batch.k_cache, batch.v_cache, batch.block_table, None,
                               batch.context_lens, cfg.scale, ks, vs, out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle.decode_attention_mq_fp8(inputs.as_u16(q), inputs.as_u8(batch.k_cache), inputs.as_u8(batch.v_cache),
                                         batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                         ks, vs, num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size,
                                         strides=batch.strides)
    assert_parity(out.reshape(B * Sq, Hq, D), ref.out.reshape(B * Sq, Hq, D), what=f"{cfg.name} Sq={Sq}")


def test_fused_step_mq_over_8bit_cache():
    cfg = C("mq8-step", 32, 8, 128, 16, (G(12, 4, 2600),), seed=97, pool_fill=0.85)
    Sq, ks, vs = 4, 1.0 / 32, 1.0 / 32
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=True), ks, vs)
    sh = binding.shape_of(batch)
    g = torch.Generator(device="cuda").manual_seed(8)
    q = torch.randn((cfg.batch, Sq, 32, 128), generator=g, device="cuda").to(torch.bfloat16)
    k_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    v_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    lens = batch.context_lens
    positions = (lens - Sq).contiguous()
    k_ref, v_ref = inputs.as_u8(batch.k_cache).copy(), inputs.as_u8(batch.v_cache).copy()
    table = batch.block_table.cpu().numpy()
    for i in range(Sq):
        oracle.kv_append_fp8(inputs.as_u16(k_new[:, i].contiguous()), inputs.as_u16(v_new[:, i].contiguous()), k_ref,
                             v_ref, table, (positions + i).cpu().numpy(), ks, vs, block_size=16, strides=batch.strides)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_step_mq_fp8(sh, q, k_new, v_new, batch.k_cache, batch.v_cache, batch.block_table, positions, lens,
                               cfg.scale, ks, vs, out, ws)
    assert binding.workspace_status(ws) == 0
    assert np.array_equal(inputs.as_u8(batch.k_cache), k_ref) and np.array_equal(inputs.as_u8(batch.v_cache), v_ref)
    ref = oracle.decode_attention_mq_fp8(inputs.as_u16(q), k_ref, v_ref, table, lens.cpu().numpy(), cfg.scale, ks, vs,
                                         num_kv_heads=8, block_size=16, strides=batch.strides)
    assert_parity(out.reshape(-1, 32, 128), ref.out.reshape(-1, 32, 128), what="fused mq step, 8-bit cache")


def run_case_8bit(cfg, Sq, seed, ks=1.0 / 32, vs=0.04):
    b16 = inputs.make_batch(cfg, "cuda", poison=True, table_pad=2**31 - 1)
    batch = inputs.to_e4m3_pool(b16, ks, vs)
    B, Hq, D = cfg.batch, cfg.num_q_heads, cfg.head_dim
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = (torch.randn((B, Sq, Hq, D), generator=g, device="cuda") * cfg.sigma).to(torch.bfloat16)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_step_mq_fp8(sh, q, None, None, batch.k_cache, batch.v_cache, batch.block_table, None,
                               batch.context_lens, cfg.scale, ks, vs, out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle.decode_attention_mq_fp8(inputs.as_u16(q), inputs.as_u8(batch.k_cache), inputs.as_u8(batch.v_cache),
                                         batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                         ks, vs, num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size,
                                         strides=batch.strides)
    assert_parity(out.reshape(B * Sq, Hq, D), ref.out.reshape(B * Sq, Hq, D), what=f"{cfg.name} Sq={Sq} (8-bit cache)")
    return batch, q, out


@pytest.mark.parametrize("cfg,Sq", [c for c in CHUNK_CASES if c[0].name in
                                    ("ck-g4-sq5", "ck-g4-sq16", "ck-g5-sq7-bs32", "ck-g1-sq100-bs128", "ck-token-major",
                                     "ck-split-g2", "ck-g4-sq10-short", "ck-g8-sq16-bs32")],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_prefill_chunk_over_8bit_cache_on_the_two_cta_kernel(cfg, Sq):
    """Up to 128 score columns over the 8-bit cache run the one-CTA-per-SM kernel's one-tile mode by default (its idle
    warps widen the codes); the kernel with two CTAs per SM, which serves more columns, stays selectable for these
    shapes and must agree with the oracle too."""
    binding.set_tuning(chunk_two_tiles=1)
    try:
        run_case_8bit(cfg, Sq, seed=cfg.seed)
    finally:
        binding.set_tuning(chunk_two_tiles=2)


@pytest.mark.parametrize("cfg,Sq", [c for c in CHUNK_CASES if c[0].head_dim == 128],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_prefill_chunk_over_8bit_cache(cfg, Sq):
    """More than 16 score columns over E4M3 caches: the tcgen05 chunk kernel with the stages widened to f16 in
    shared memory (17 columns up to several row tiles, every block size, split sequences)."""
    batch, q, out = run_case_8bit(cfg, Sq, seed=cfg.seed)
    out2 = torch.full_like(out, float("nan"))
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    binding.decode_step_mq_fp8(sh, q, None, None, batch.k_cache, batch.v_cache, batch.block_table, None,
                               batch.context_lens, cfg.scale, 1.0 / 32, 0.04, out2, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))                    # run-to-run bitwise


def test_fused_step_prefill_chunk_over_8bit_cache():
    """The quantising append of a 40-token chunk (bit-exact over the whole pool) fused into the first launch, seen by
    the attention of the same call."""
    cfg = C("ck8-step", 32, 8, 128, 16, (G(6, 40, 1500),), seed=121, pool_fill=0.85)
    Sq, ks, vs = 40, 1.0 / 32, 1.0 / 32
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=True), ks, vs)
    sh = binding.shape_of(batch)
    g = torch.Generator(device="cuda").manual_seed(10)
    q = torch.randn((cfg.batch, Sq, 32, 128), generator=g, device="cuda").to(torch.bfloat16)
    k_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    v_new = torch.randn((cfg.batch, Sq, 8, 128), generator=g, device="cuda").to(torch.bfloat16)
    lens = batch.context_lens
    positions = (lens - Sq).contiguous()
    k_ref, v_ref = inputs.as_u8(batch.k_cache).copy(), inputs.as_u8(batch.v_cache).copy()
    table = batch.block_table.cpu().numpy()
    for i in range(Sq):
        oracle.kv_append_fp8(inputs.as_u16(k_new[:, i].contiguous()), inputs.as_u16(v_new[:, i].contiguous()), k_ref,
                             v_ref, table, (positions + i).cpu().numpy(), ks, vs, block_size=16, strides=batch.strides)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_step_mq_fp8(sh, q, k_new, v_new, batch.k_cache, batch.v_cache, batch.block_table, positions, lens,
                               cfg.scale, ks, vs, out, ws)
    assert binding.workspace_status(ws) == 0 and binding.last_launch_count() == 3
    assert np.array_equal(inputs.as_u8(batch.k_cache), k_ref) and np.array_equal(inputs.as_u8(batch.v_cache), v_ref)
    ref = oracle.decode_attention_mq_fp8(inputs.as_u16(q), k_ref, v_ref, table, lens.cpu().numpy(), cfg.scale, ks, vs,
                                         num_kv_heads=8, block_size=16, strides=batch.strides)
    assert_parity(out.reshape(-1, 32, 128), ref.out.reshape(-1, 32, 128), what="fused chunk step, 8-bit cache")
