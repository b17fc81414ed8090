"""Seeded random shapes and length mixes against the oracle: bf16, 8-bit cache, several query tokens, prefill chunks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs
from util import MAX_ABS_TOL, MEAN_ABS_TOL, bf16_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def assert_close(out_gpu, ref, what):
    """The parity tolerance, plus half a bf16 unit in the last place of the expected value: with contexts
    of two or three tokens an output is as large as a single V entry (up to 4 or 5 here), and rounding
    such a value to bf16 alone moves it by up to 2^-8 of its magnitude."""
    got = bf16_to_f64(out_gpu)
    assert not np.isnan(ref).any() and not np.isnan(got).any(), what
    err = np.abs(got - ref)
    excess = err - np.abs(ref) * 2.0 ** -8
    assert excess.max() <= MAX_ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert err.mean() <= MEAN_ABS_TOL, f"{what}: mean abs err {err.mean():.3e}"


def draw_case(seed):
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128, 128]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 5, 7, 8, 12, 16]))
    bs = int(rng.choice([16, 16, 32, 64, 128]))
    B = int(rng.integers(1, 24))
    kinds = rng.integers(0, 4, B)
    lens = np.where(kinds == 0, rng.integers(0, 4, B),
                    np.where(kinds == 1, rng.integers(1, 200, B),
                             np.where(kinds == 2, rng.integers(200, 3000, B), rng.integers(3000, 12000, B))))
    if rng.random() < 0.3:
        lens[rng.integers(0, B)] = int(rng.choice([63, 64, 65, 127, 128, 129, 255, 256, 257, 8191, 8192, 8193]))
    layout = "token_major" if rng.random() < 0.25 else "head_major"
    mode = "bf16"
    if D == 128 and rng.random() < 0.3:
        mode = "fp8"
    elif rng.random() < 0.35:
        mode = "mq"
    Sq = 1
    if mode == "mq":
        choices = [s for s in (2, 3, 4, 8, 16) if s * G <= 16]
        if not choices:
            mode = "bf16"
        else:
            Sq = int(rng.choice(choices))
            if D == 128 and rng.random() < 0.4:
                mode = "mq8"
    cfg = inputs.DecodeConfig(f"fuzz{seed}", Hkv * G, Hkv, D, bs,
                              (inputs.LengthGroup(B, int(lens.min()), int(lens.max()), "fixed", tuple(int(x) for x in lens)),),
                              seed=2000 + seed, pool_fill=float(rng.choice([1.0, 0.9, 0.6])), layout=layout,
                              shuffle_batch=False)
    return cfg, mode, Sq


@pytest.mark.parametrize("seed", range(64))
def test_random_case(seed):
    cfg, mode, Sq = draw_case(seed)
    batch = inputs.make_batch(cfg, "cuda", poison=True, table_pad=-7)
    kw = dict(num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size, strides=batch.strides)
    table, lens = batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy()
    if mode == "fp8":
        ks, vs = 1.0 / 16, 1.0 / 64
        b8 = inputs.to_e4m3_pool(batch, ks, vs)
        sh = binding.shape_of(b8)
        ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
        out = torch.full_like(batch.q, float("nan"))
        binding.decode_attention_fp8(sh, b8.q, b8.k_cache, b8.v_cache, b8.block_table, b8.context_lens, cfg.scale, ks, vs,
                                     out, ws)
        ref = oracle.decode_attention_fp8(inputs.as_u16(b8.q), inputs.as_u8(b8.k_cache), inputs.as_u8(b8.v_cache), table,
                                          lens, cfg.scale, ks, vs, **kw).out
    elif mode == "mq8":
        ks, vs = 1.0 / 16, 1.0 / 64
        b8 = inputs.to_e4m3_pool(batch, ks, vs)
        g = torch.Generator(device="cuda").manual_seed(seed)
        q = torch.randn((cfg.batch, Sq, cfg.num_q_heads, cfg.head_dim), generator=g, device="cuda").to(torch.bfloat16)
        sh = binding.shape_of(b8)
        ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
        out = torch.full_like(q, float("nan"))
        binding.decode_step_mq_fp8(sh, q, None, None, b8.k_cache, b8.v_cache, b8.block_table, None, b8.context_lens,
                                   cfg.scale, ks, vs, out, ws)
        ref = oracle.decode_attention_mq_fp8(inputs.as_u16(q), inputs.as_u8(b8.k_cache), inputs.as_u8(b8.v_cache), table,
                                             lens, cfg.scale, ks, vs, **kw).out
        out, ref = out.reshape(-1, cfg.num_q_heads, cfg.head_dim), ref.reshape(-1, cfg.num_q_heads, cfg.head_dim)
    elif mode == "mq":
        g = torch.Generator(device="cuda").manual_seed(seed)
        q = torch.randn((cfg.batch, Sq, cfg.num_q_heads, cfg.head_dim), generator=g, device="cuda").to(torch.bfloat16)
        sh = binding.shape_of(batch)
        ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
        out = torch.full_like(q, float("nan"))
        binding.decode_attention_mq(sh, q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens, cfg.scale,
                                    out, ws)
        ref = oracle.decode_attention_mq(inputs.as_u16(q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache), table,
                                         lens, cfg.scale, **kw).out
        out, ref = out.reshape(-1, cfg.num_q_heads, cfg.head_dim), ref.reshape(-1, cfg.num_q_heads, cfg.head_dim)
    else:
        sh = binding.shape_of(batch)
        ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
        out = torch.full_like(batch.q, float("nan"))
        binding.decode_attention(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                                 cfg.scale, out, ws)
        ref = oracle.decode_attention(inputs.as_u16(batch.q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
                                      table, lens, cfg.scale, **kw).out
    assert binding.workspace_status(ws) == 0
    assert_close(out, ref, what=f"{cfg.name} {mode} Sq={Sq} G={cfg.num_q_heads // cfg.num_kv_heads} D={cfg.head_dim} "
                                 f"bs={cfg.block_size} {cfg.layout}")


def draw_chunk_case(seed):
    """Random prefill chunks: more than 8 score columns per (sequence, kv head), i.e. the two row-layout
    kernels; contexts shorter than, equal to and far longer than the chunk."""
    rng = np.random.default_rng(5000 + seed)
    D = int(rng.choice([64, 128, 128]))
    Hkv = int(rng.choice([1, 2, 2, 4]))
    G = int(rng.choice([1, 2, 3, 4, 5, 8, 16]))
    bs = int(rng.choice([16, 16, 32, 64, 128, 256]))
    B = int(rng.integers(1, 6))
    Sq = int(rng.choice([2, 3, 5, 8, 16, 17, 31, 32, 33, 48, 64, 65, 80]))
    while Sq * G <= 8:
        Sq *= 2
    kinds = rng.integers(0, 4, B)
    lens = np.where(kinds == 0, rng.integers(0, Sq + 2, B),                  # shorter than / about the chunk
                    np.where(kinds == 1, Sq + rng.integers(0, 3, B),         # a fresh prompt: context = chunk
                             np.where(kinds == 2, rng.integers(Sq, 700, B), rng.integers(700, 6000, B))))
    # keep the oracle's work bounded: rows x tokens
    while B * Sq * Hkv * G * max(1, int(lens.mean())) > 6_000_000:
        lens = np.maximum(lens // 2, 1)
    layout = "token_major" if rng.random() < 0.25 else "head_major"
    cfg = inputs.DecodeConfig(f"chunkfuzz{seed}", Hkv * G, Hkv, D, bs,
                              (inputs.LengthGroup(B, int(lens.min()), int(lens.max()), "fixed", tuple(int(x) for x in lens)),),
                              seed=6000 + seed, pool_fill=float(rng.choice([1.0, 0.8])), layout=layout,
                              shuffle_batch=False)
    return cfg, Sq


@pytest.mark.parametrize("seed", range(32))
def test_random_chunk_case(seed):
    cfg, Sq = draw_chunk_case(seed)
    batch = inputs.make_batch(cfg, "cuda", poison=True, table_pad=-7)
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = torch.randn((cfg.batch, Sq, cfg.num_q_heads, cfg.head_dim), generator=g, device="cuda").to(torch.bfloat16)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    binding.decode_attention_mq(sh, q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens, cfg.scale,
                                out, ws)
    assert binding.workspace_status(ws) == 0
    ref = oracle.decode_attention_mq(inputs.as_u16(q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
                                     batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), cfg.scale,
                                     num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size, strides=batch.strides).out
    assert_close(out.reshape(-1, cfg.num_q_heads, cfg.head_dim), ref.reshape(-1, cfg.num_q_heads, cfg.head_dim),
                 what=f"{cfg.name} Sq={Sq} G={cfg.num_q_heads // cfg.num_kv_heads} D={cfg.head_dim} bs={cfg.block_size} "
                      f"{cfg.layout} lens={batch.context_lens.cpu().tolist()}")
