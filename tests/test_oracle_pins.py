"""Pins of the fp64 CPU oracle against things other than itself.

The paper prints no worked attention values, so the oracle is pinned by: a structurally
different brute force (gather to contiguous, heads repeated, no max-subtraction), a library
softmax attention in fp64, closed forms, and the invariants of softmax attention over a
paged cache.  Each pin is chosen to break under one plausible mistake (head mapping, scale,
slot/block indexing, transposed operand, missing normalisation, tail handling).
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import inputs


def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    """Exact widening done with numpy views (independent of the oracle's C decoder)."""
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    return inputs.as_u16(torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def gather_contiguous(batch, b):
    """K, V of sequence b as float64 [T, Hkv, D] via explicit per-token indexing."""
    cfg = batch.cfg
    T = int(batch.context_lens[b])
    bs = cfg.block_size
    k4 = bf16_to_f64(inputs.as_u16(batch.k_cache))
    v4 = bf16_to_f64(inputs.as_u16(batch.v_cache))
    K = np.empty((T, cfg.num_kv_heads, cfg.head_dim))
    V = np.empty_like(K)
    for t in range(T):
        blk = int(batch.block_table[b, t // bs])
        if cfg.layout == "head_major":
            K[t], V[t] = k4[blk, :, t % bs, :], v4[blk, :, t % bs, :]
        else:
            K[t], V[t] = k4[blk, t % bs, :, :], v4[blk, t % bs, :, :]
    return K, V


def run_oracle(batch, scale=None, pairs=None, context_lens=None):
    cfg = batch.cfg
    return oracle.decode_attention(
        inputs.as_u16(batch.q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
        batch.block_table.numpy(), (batch.context_lens if context_lens is None else context_lens).numpy(),
        cfg.scale if scale is None else scale, num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size,
        strides=batch.strides, pairs=pairs)


SMALL = [
    inputs.CONFIGS["cfg0"],
    inputs.replace(inputs.CONFIGS["cfg0"], layout="token_major", seed=10, name="cfg0-token-major"),
    inputs.DecodeConfig("g5", 10, 2, 128, 32, (inputs.LengthGroup(3, 1, 150),), seed=11, pool_fill=0.8),
    inputs.DecodeConfig("mha", 4, 4, 64, 16, (inputs.LengthGroup(3, 1, 70),), seed=12),
    inputs.DecodeConfig("mqa", 8, 1, 64, 16, (inputs.LengthGroup(2, 5, 40),), seed=13),
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_brute_force_without_max_subtraction(cfg):
    batch = inputs.make_batch(cfg, poison=True)
    res = run_oracle(batch, scale=0.37)                       # scale != 1/sqrt(D): catches a hard-coded scale
    G = cfg.num_q_heads // cfg.num_kv_heads
    qf = bf16_to_f64(inputs.as_u16(batch.q))
    for b in range(cfg.batch):
        K, V = gather_contiguous(batch, b)
        Kr, Vr = np.repeat(K, G, axis=1), np.repeat(V, G, axis=1)          # [T, Hq, D], heads repeated
        s = 0.37 * np.einsum("hd,thd->ht", qf[b], Kr)
        e = np.exp(s)                                                       # no max-subtraction
        w = e / e.sum(axis=1, keepdims=True)
        ref = np.einsum("ht,thd->hd", w, Vr)
        np.testing.assert_allclose(res.out[b], ref, rtol=0, atol=1e-12)
        np.testing.assert_allclose(res.lse[b], np.log(e.sum(axis=1)), rtol=0, atol=1e-12)
    assert not np.isnan(res.out).any()                                      # poison never read
    np.testing.assert_allclose(res.wsum, 1.0, rtol=0, atol=1e-12)           # weights sum to 1


@pytest.mark.parametrize("cfg", SMALL[:3], ids=lambda c: c.name)
def test_library_sdpa_fp64(cfg):
    batch = inputs.make_batch(cfg, poison=True)
    res = run_oracle(batch)
    G = cfg.num_q_heads // cfg.num_kv_heads
    qf = torch.from_numpy(bf16_to_f64(inputs.as_u16(batch.q)))
    for b in range(cfg.batch):
        K, V = gather_contiguous(batch, b)
        Kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(G, dim=0)   # [Hq, T, D]
        Vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(G, dim=0)
        ref = torch.nn.functional.scaled_dot_product_attention(
            qf[b].unsqueeze(1), Kt, Vt, scale=cfg.scale)                        # [Hq, 1, D]
        np.testing.assert_allclose(res.out[b], ref.squeeze(1).numpy(), rtol=0, atol=1e-12)


def test_closed_form_two_tokens():
    """Scores 0 and 1 give weights 1/(1+e), e/(1+e) (softmax by hand)."""
    cfg = inputs.DecodeConfig("two", 1, 1, 64, 16, (inputs.LengthGroup(1, 2, 2, "fixed", (2,)),), seed=5)
    batch = inputs.make_batch(cfg, poison=True)
    blk = int(batch.block_table[0, 0])
    q = torch.zeros(64); q[3] = 2.0
    k0 = torch.zeros(64); k1 = torch.zeros(64); k1[3] = 4.0; k1[7] = 100.0      # q.k0 = 0, q.k1 = 8
    batch.q[0, 0] = q.to(torch.bfloat16)
    batch.k_cache[blk, 0, 0] = k0.to(torch.bfloat16)
    batch.k_cache[blk, 0, 1] = k1.to(torch.bfloat16)
    res = run_oracle(batch, scale=0.125)                                         # scores 0 and 1
    v = bf16_to_f64(inputs.as_u16(batch.v_cache))[blk, 0]
    ref = (v[0] + math.e * v[1]) / (1.0 + math.e)
    np.testing.assert_allclose(res.out[0, 0], ref, rtol=0, atol=1e-14)
    assert abs(res.lse[0, 0] - math.log(1.0 + math.e)) < 1e-14


def test_context_one_returns_value_exactly():
    cfg = inputs.DecodeConfig("one", 8, 2, 64, 16, (inputs.LengthGroup(3, 1, 1, "fixed", (1, 1, 1)),), seed=6)
    batch = inputs.make_batch(cfg, poison=True)
    res = run_oracle(batch)
    v = bf16_to_f64(inputs.as_u16(batch.v_cache))
    for b in range(3):
        blk = int(batch.block_table[b, 0])
        for hq in range(8):
            assert np.array_equal(res.out[b, hq], v[blk, hq // 4, 0])           # bit-exact


def test_identical_keys_and_zero_query_give_mean_of_values():
    cfg = inputs.DecodeConfig("mean", 4, 2, 64, 16, (inputs.LengthGroup(2, 37, 53),), seed=7)
    batch = inputs.make_batch(cfg, poison=False)
    same = batch.k_cache[0, :, 0, :].clone()
    batch.k_cache[:] = same.view(1, 2, 1, 64)                                    # every key of a head identical
    res = run_oracle(batch)
    batch2 = inputs.make_batch(cfg, poison=True)
    batch2.q.zero_()                                                             # q = 0: all scores equal
    res2 = run_oracle(batch2)
    for bt, rs in ((batch, res), (batch2, res2)):
        for b in range(2):
            _, V = gather_contiguous(bt, b)
            mean = V.mean(axis=0)                                                # [Hkv, D]
            for hq in range(4):
                np.testing.assert_allclose(rs.out[b, hq], mean[hq // 2], rtol=0, atol=1e-13)


def test_block_permutation_is_bit_identical():
    cfg = inputs.CONFIGS["cfg0"]
    batch = inputs.make_batch(cfg, poison=True)
    res = run_oracle(batch)
    g = torch.Generator().manual_seed(99)
    perm = torch.randperm(batch.num_blocks, generator=g)                         # new id of old block i
    k2, v2 = torch.empty_like(batch.k_cache), torch.empty_like(batch.v_cache)
    k2[perm], v2[perm] = batch.k_cache, batch.v_cache
    t2 = batch.block_table.clone()
    ok = t2 >= 0
    t2[ok] = perm[t2[ok].long()].to(torch.int32)
    res2 = oracle.decode_attention(
        inputs.as_u16(batch.q), inputs.as_u16(k2), inputs.as_u16(v2), t2.numpy(),
        batch.context_lens.numpy(), cfg.scale, num_kv_heads=cfg.num_kv_heads,
        block_size=cfg.block_size, strides=batch.strides)
    assert np.array_equal(res.out, res2.out) and np.array_equal(res.lse, res2.lse)


def test_key_shift_invariance():
    """Adding one vector to every key changes every score of a head by the same amount."""
    cfg = inputs.DecodeConfig("shift", 4, 2, 64, 16, (inputs.LengthGroup(2, 20, 45),), seed=8)
    batch = inputs.make_batch(cfg, poison=False)
    gen = torch.Generator().manual_seed(3)
    ki = torch.randint(-8, 9, batch.k_cache.shape, generator=gen).float()       # small integers: exact in bf16
    qi = torch.randint(-4, 5, batch.q.shape, generator=gen).float()
    c = torch.randint(-8, 9, (64,), generator=gen).float()
    batch.q[:] = qi.to(torch.bfloat16)
    batch.k_cache[:] = ki.to(torch.bfloat16)
    res = run_oracle(batch, scale=1.0 / 64)
    batch.k_cache[:] = (ki + c).to(torch.bfloat16)
    res2 = run_oracle(batch, scale=1.0 / 64)
    np.testing.assert_allclose(res.out, res2.out, rtol=0, atol=1e-12)
    shift = (bf16_to_f64(inputs.as_u16(batch.q)) @ c.double().numpy()) / 64
    np.testing.assert_allclose(res2.lse - res.lse, shift, rtol=0, atol=1e-12)


def test_partition_merge_equals_unpartitioned():
    """Log-sum-exp merge of the oracle's results over a partition of [0, T) (the split-KV identity)."""
    cfg = inputs.DecodeConfig("part", 8, 2, 64, 16, (inputs.LengthGroup(1, 200, 200),), seed=9)
    batch = inputs.make_batch(cfg, poison=True)
    full = run_oracle(batch)
    T = int(batch.context_lens[0])
    cuts = [0, 48, 112, T]                                                        # block-aligned cuts
    outs, lses = [], []
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        # the sub-range [lo, hi) as its own sequence: drop the first lo/bs blocks of the table
        t2 = torch.roll(batch.block_table, -(lo // 16), dims=1)
        r = oracle.decode_attention(
            inputs.as_u16(batch.q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache),
            t2.numpy(), np.array([hi - lo], dtype=np.int32), cfg.scale, num_kv_heads=2,
            block_size=16, strides=batch.strides)
        outs.append(r.out[0]); lses.append(r.lse[0])
    lses = np.stack(lses); outs = np.stack(outs)                                  # [C, Hq], [C, Hq, D]
    M = lses.max(axis=0)
    w = np.exp(lses - M)
    merged = (w[:, :, None] * outs).sum(axis=0) / w.sum(axis=0)[:, None]
    np.testing.assert_allclose(merged, full.out[0], rtol=0, atol=1e-13)
    np.testing.assert_allclose(M + np.log(w.sum(axis=0)), full.lse[0], rtol=0, atol=1e-12)


def test_zero_length_and_pairs_subset():
    cfg = inputs.DecodeConfig("z", 4, 2, 64, 16, (inputs.LengthGroup(3, 9, 30),), seed=14)
    batch = inputs.make_batch(cfg, poison=True)
    lens = batch.context_lens.clone(); lens[1] = 0
    res = run_oracle(batch, context_lens=lens)
    assert np.array_equal(res.out[1], np.zeros((4, 64))) and np.all(np.isneginf(res.lse[1]))
    sub = run_oracle(batch, context_lens=lens, pairs=np.array([[2, 3], [0, 1]], dtype=np.int32))
    assert np.array_equal(sub.out[2, 3], res.out[2, 3]) and np.array_equal(sub.out[0, 1], res.out[0, 1])
    assert np.isnan(sub.out[0, 0]).all()


def test_bad_table_entry_is_reported():
    cfg = inputs.DecodeConfig("bad", 2, 1, 64, 16, (inputs.LengthGroup(1, 40, 40),), seed=15)
    batch = inputs.make_batch(cfg)
    batch.block_table[0, 1] = batch.num_blocks
    with pytest.raises(ValueError):
        run_oracle(batch)


# ---------------------------------------------------------------- KV append
@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_kv_append_against_numpy_indexing(layout):
    cfg = inputs.DecodeConfig("app", 8, 2, 64, 16, (inputs.LengthGroup(5, 1, 80),), seed=16, pool_fill=0.7,
                              layout=layout)
    batch = inputs.make_batch(cfg, poison=True)
    lens = batch.context_lens.clone()
    lens[0] = 32                                                                  # position on a block boundary
    batch = inputs.make_batch(cfg, poison=True, context_lens=lens)
    k0, v0 = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    k1, v1 = k0.copy(), v0.copy()
    n = oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k1, v1,
                         batch.block_table.numpy(), batch.context_lens.numpy(), block_size=16,
                         strides=batch.strides)
    assert n == 5
    kn, vn = inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new)
    for b in range(5):
        pos = int(batch.context_lens[b]); blk = int(batch.block_table[b, pos // 16])
        if layout == "head_major":
            k0[blk, :, pos % 16, :], v0[blk, :, pos % 16, :] = kn[b], vn[b]
        else:
            k0[blk, pos % 16, :, :], v0[blk, pos % 16, :, :] = kn[b], vn[b]
    assert np.array_equal(k0, k1) and np.array_equal(v0, v1)                      # incl. every untouched word


def test_kv_append_skips_out_of_range():
    cfg = inputs.DecodeConfig("app2", 4, 2, 64, 16, (inputs.LengthGroup(3, 5, 20),), seed=17)
    batch = inputs.make_batch(cfg)
    k1, v1 = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    pos = np.array([-1, batch.max_blocks_per_seq * 16, 3], dtype=np.int32)
    n = oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k1, v1,
                         batch.block_table.numpy(), pos, block_size=16, strides=batch.strides)
    assert n == 1


def test_append_then_attend_context_one_more():
    """After appending at T, attention over T + 1 tokens with q.k_new dominating returns ~v_new."""
    cfg = inputs.DecodeConfig("aa", 2, 1, 64, 16, (inputs.LengthGroup(1, 31, 31),), seed=18)
    batch = inputs.make_batch(cfg, poison=True)
    batch.k_new[0, 0] = (batch.q[0, 0].float() * 60).to(torch.bfloat16)          # huge score for the new token
    k1, v1 = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k1, v1,
                     batch.block_table.numpy(), batch.context_lens.numpy(), block_size=16,
                     strides=batch.strides)
    r = oracle.decode_attention(inputs.as_u16(batch.q), k1, v1, batch.block_table.numpy(),
                                batch.context_lens.numpy() + 1, 1.0, num_kv_heads=1, block_size=16,
                                strides=batch.strides)
    vnew = bf16_to_f64(inputs.as_u16(batch.v_new))[0, 0]
    np.testing.assert_allclose(r.out[0, 0], vnew, rtol=0, atol=1e-9)


def test_multi_query_oracle_is_bottom_right_causal_attention():
    """S_q > 1: against a library softmax attention in fp64 with an explicit causal mask aligned to the
    end of the sequence, on gathered contiguous K / V with heads repeated."""
    rng = np.random.default_rng(11)
    B, Sq, Hq, Hkv, D, bs, NB = 3, 3, 4, 2, 8, 4, 12
    lens = np.array([9, 3, 14], dtype=np.int32)                 # the second sequence is nothing but its queries
    table = np.stack([rng.permutation(NB)[:4] for _ in range(B)]).astype(np.int32)
    to_bits = lambda x: torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    from_bits = lambda u: torch.from_numpy(u.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64)
    k = to_bits(rng.standard_normal((NB, Hkv, bs, D)))
    v = to_bits(rng.standard_normal((NB, Hkv, bs, D)))
    q = to_bits(rng.standard_normal((B, Sq, Hq, D)))
    got = oracle.decode_attention_mq(q, k, v, table, lens, 0.4, num_kv_heads=Hkv, block_size=bs,
                                     strides=(Hkv * bs * D, bs * D, D))
    kf, vf, qf = from_bits(k), from_bits(v), from_bits(q)
    for b in range(B):
        T = int(lens[b])
        blocks = torch.from_numpy(table[b, :(T + bs - 1) // bs].astype(np.int64))
        kk = kf[blocks].permute(1, 0, 2, 3).reshape(Hkv, -1, D)[:, :T].repeat_interleave(Hq // Hkv, 0)   # [Hq, T, D]
        vv = vf[blocks].permute(1, 0, 2, 3).reshape(Hkv, -1, D)[:, :T].repeat_interleave(Hq // Hkv, 0)
        mask = torch.ones(Sq, T, dtype=torch.bool).tril(diagonal=T - Sq)                                # query i sees t <= T - Sq + i
        want = torch.nn.functional.scaled_dot_product_attention(qf[b].permute(1, 0, 2), kk, vv, attn_mask=mask, scale=0.4)
        assert np.allclose(got.out[b], want.permute(1, 0, 2).numpy(), atol=1e-12)
    assert np.allclose(got.wsum, 1.0, atol=1e-12)
    # S_q = 1 is the one-query operator itself
    one = oracle.decode_attention_mq(q[:, -1:], k, v, table, lens, 0.4, num_kv_heads=Hkv, block_size=bs,
                                     strides=(Hkv * bs * D, bs * D, D))
    assert np.array_equal(one.out[:, 0], got.out[:, -1])
