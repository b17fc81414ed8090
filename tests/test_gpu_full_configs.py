"""Full-size workloads (the benchmark's configurations and launch shape) vs the oracle.

Every output of every configuration is compared: all B * Hq * D values, no sampling.  The larger
pools do not go to the host in one piece; the oracle takes the sequences in consecutive runs, each
with a host copy of just that run's blocks.  The append of the fragmentation workload is compared
word for word over the entire pool.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs
from util import assert_parity, gpu_attention, oracle_attention, oracle_attention_every_sequence

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def test_cfg1_every_output():
    batch = inputs.make_batch(inputs.CONFIGS["cfg1"], "cuda", poison=True)
    out = gpu_attention(batch)
    mx, mean = assert_parity(out, oracle_attention(batch).out, what="cfg1")
    print(f"cfg1 max abs {mx:.3e} mean abs {mean:.3e}")


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4"])
def test_large_config_every_output(name):
    cfg = inputs.CONFIGS[name]
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    out = gpu_attention(batch)
    ref = oracle_attention_every_sequence(batch)
    assert ref.shape == (cfg.batch, cfg.num_q_heads, cfg.head_dim)
    mx, mean = assert_parity(out, ref, what=name)
    print(f"{name} all {ref.size} outputs: max abs {mx:.3e} mean abs {mean:.3e}")
    # property that holds at any size: every output lies in the convex hull of its V values
    step = 1 << 13                                                                      # blocks per chunk
    bound = max(float(torch.nan_to_num(batch.v_cache[s:s + step].float(), nan=0.0).abs().max())
                for s in range(0, batch.num_blocks, step))
    assert float(out.float().abs().max()) <= bound * 1.01

    if name == "cfg4":
        # one-token append for every sequence at position T_b: whole pool compared word for word
        sh = binding.shape_of(batch)
        k_ref, v_ref = inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache)      # host copies
        n = oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k_ref, v_ref,
                             batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(),
                             block_size=cfg.block_size, strides=batch.strides)
        assert n == cfg.batch
        binding.kv_append(sh, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                          batch.context_lens)
        torch.cuda.synchronize()
        k_ref_t = torch.from_numpy(k_ref.view(np.int16))
        v_ref_t = torch.from_numpy(v_ref.view(np.int16))
        step = 1 << 14                                                                  # blocks per compare chunk
        for s in range(0, batch.num_blocks, step):
            assert torch.equal(batch.k_cache[s:s + step].view(torch.int16).cpu(), k_ref_t[s:s + step])
            assert torch.equal(batch.v_cache[s:s + step].view(torch.int16).cpu(), v_ref_t[s:s + step])
        # and the serving order: attention over T_b + 1 tokens sees the appended token
        lens1 = (batch.context_lens + 1).contiguous()
        out1 = gpu_attention(batch, context_lens=lens1)
        ref1 = oracle_attention_every_sequence(batch, context_lens=lens1)
        assert_parity(out1, ref1, what="cfg4 after append")


@pytest.mark.parametrize("name", ["cfg1", "cfg3"])
def test_fp8_cache_full_size_every_output(name):
    """The 8-bit cache path at benchmark size and launch shape: fused step, every output."""
    cfg = inputs.CONFIGS[name]
    ks, vs = 1.0 / 32, 1.0 / 32
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=True), ks, vs)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    out = torch.full_like(batch.q, float("nan"))
    lens1 = (batch.context_lens + 1).contiguous()
    binding.decode_step_fp8(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                            batch.context_lens, lens1, cfg.scale, ks, vs, out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle_attention_every_sequence(batch, context_lens=lens1, kv8=(ks, vs))      # on the pool after the append
    mx, mean = assert_parity(out, ref, what=name + " fp8")
    print(f"{name} fp8 all {ref.size} outputs: max abs {mx:.3e} mean abs {mean:.3e}")


def test_very_long_context_next_to_very_short_ones():
    """One 400 K-token sequence (50 chunks per kv head at the largest chunk size, two rounds of the
    merge's 32-chunk batches for nobody, but a deep partial list) beside sequences of 1 and 40 tokens."""
    cfg = inputs.DecodeConfig("long", 32, 8, 128, 16, (inputs.LengthGroup(3, 1, 400_000, "fixed", (400_000, 1, 40)),),
                              seed=95, shuffle_batch=False)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    out = gpu_attention(batch)
    assert torch.isfinite(out.float()).all()
    pairs = np.array([(0, 0), (0, 13), (0, 31), (1, 5), (2, 0), (2, 31)], dtype=np.int32)
    ref = oracle.decode_attention(inputs.as_u16(batch.q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
                                  batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                  num_kv_heads=8, block_size=16, strides=batch.strides, pairs=pairs)
    got = out.cpu().double().numpy()
    for b, h in pairs:
        err = np.abs(got[b, h] - ref.out[b, h])
        assert err.max() <= 1e-2 and err.mean() <= 1e-3, (b, h, err.max())


@pytest.mark.parametrize("Sq", [4, 16, 64], ids=["16-columns", "64-columns", "256-columns"])
def test_prefill_chunk_full_size_every_output(Sq):
    """Several query tokens per sequence at benchmark size and launch shape (cfg1 with the chunk added to every
    context): the 16-column row-layout kernel and the tcgen05 chunk kernel in its one-tile and its two-tile mode;
    every row of every sequence against the oracle."""
    base = inputs.CONFIGS["cfg1"]
    cfg = inputs.replace(base, groups=tuple(inputs.replace(g, lo=g.lo + Sq, hi=g.hi + Sq) for g in base.groups))
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    B, Hq, D, bs = cfg.batch, cfg.num_q_heads, cfg.head_dim, cfg.block_size
    gen = torch.Generator(device="cuda").manual_seed(77)
    q = torch.randn((B, Sq, Hq, D), generator=gen, device="cuda").to(torch.bfloat16)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_attention_mq(sh, q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens, cfg.scale,
                                out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle.decode_attention_mq(inputs.as_u16(q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
                                     batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                     num_kv_heads=cfg.num_kv_heads, block_size=bs, strides=batch.strides)
    assert ref.out.shape == (B, Sq, Hq, D)
    mx, mean = assert_parity(out.reshape(-1, Hq, D), ref.out.reshape(-1, Hq, D), what=f"cfg1 + chunk of {Sq}")
    print(f"cfg1 with {Sq} query tokens, all {ref.out.size} outputs: max abs {mx:.3e} mean abs {mean:.3e}")


def test_small_chunk_on_the_long_context_mix_every_output():
    """cfg3 with 8 query tokens per sequence (64 score columns: the tcgen05 chunk kernel's one-tile mode) at
    benchmark size and launch shape: 115 short sequences of one to eight 128-token slots beside 13 of 32 K to 64 K
    tokens, so units of every length, split and unsplit, follow each other in every CTA.  Three launches give the
    same bits (the hand-overs between the issuing warps and the softmax threads do not depend on timing), and every
    output agrees with the oracle."""
    Sq = 8
    base = inputs.CONFIGS["cfg3"]
    cfg = inputs.replace(base, groups=tuple(inputs.replace(g, lo=g.lo + Sq, hi=g.hi + Sq) for g in base.groups))
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    B, Hq, D, bs = cfg.batch, cfg.num_q_heads, cfg.head_dim, cfg.block_size
    gen = torch.Generator(device="cuda").manual_seed(79)
    q = (torch.randn((B, Sq, Hq, D), generator=gen, device="cuda") * cfg.sigma).to(torch.bfloat16)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(3):
        out = torch.full_like(q, float("nan"))
        binding.decode_attention_mq(sh, q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens, cfg.scale,
                                    out, ws)
        assert binding.workspace_status(ws) == 0
        outs.append(out)
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
    assert torch.equal(outs[0].view(torch.int16), outs[2].view(torch.int16))
    ref = oracle.decode_attention_mq(inputs.as_u16(q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
                                     batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                     num_kv_heads=cfg.num_kv_heads, block_size=bs, strides=batch.strides)
    mx, mean = assert_parity(outs[0].reshape(-1, Hq, D), ref.out.reshape(-1, Hq, D), what="cfg3 + chunk of 8")
    print(f"cfg3 with 8 query tokens, all {ref.out.size} outputs: max abs {mx:.3e} mean abs {mean:.3e}")


@pytest.mark.parametrize("Sq", [16, 64], ids=["64-columns", "256-columns"])
def test_prefill_chunk_over_8bit_cache_full_size_every_output(Sq):
    """cfg1 with a chunk of 16 or 64 tokens per sequence over E4M3 caches (64 score columns: the one-CTA kernel's
    one-tile mode, whose spare warps widen the stages; 256 columns: two row tiles of the two-CTA kernel, stages
    widened in shared memory by warps of their own), every output against the 8-bit oracle."""
    ks, vs = 1.0 / 32, 1.0 / 32
    base = inputs.CONFIGS["cfg1"]
    cfg = inputs.replace(base, groups=tuple(inputs.replace(g, lo=g.lo + Sq, hi=g.hi + Sq) for g in base.groups))
    batch = inputs.to_e4m3_pool(inputs.make_batch(cfg, "cuda", poison=True), ks, vs)
    B, Hq, D, bs = cfg.batch, cfg.num_q_heads, cfg.head_dim, cfg.block_size
    gen = torch.Generator(device="cuda").manual_seed(78)
    q = torch.randn((B, Sq, Hq, D), generator=gen, device="cuda").to(torch.bfloat16)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_step_mq_fp8(sh, q, None, None, batch.k_cache, batch.v_cache, batch.block_table, None,
                               batch.context_lens, cfg.scale, ks, vs, out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle.decode_attention_mq_fp8(inputs.as_u16(q), inputs.as_u8(batch.k_cache), inputs.as_u8(batch.v_cache),
                                         batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                         ks, vs, num_kv_heads=cfg.num_kv_heads, block_size=bs, strides=batch.strides)
    mx, mean = assert_parity(out.reshape(-1, Hq, D), ref.out.reshape(-1, Hq, D), what=f"cfg1 + chunk of {Sq}, 8-bit cache")
    print(f"cfg1 with {Sq} query tokens over an 8-bit cache, all {ref.out.size} outputs: max abs {mx:.3e} mean abs {mean:.3e}")
