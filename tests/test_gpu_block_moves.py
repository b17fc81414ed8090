"""Paged block movement (gather / scatter / copy) on the GPU vs the oracle: bit-exact, whole pool."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def make_pool(layout, NB, Hkv, bs, D, seed):
    """(k, v, strides): bf16 device pools holding random bit patterns (NaN patterns included)."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    if layout == "head_major":
        shape, strides = (NB, Hkv, bs, D), (Hkv * bs * D, bs * D, D)
    elif layout == "token_major":
        shape, strides = (NB, bs, Hkv, D), (bs * Hkv * D, D, Hkv * D)
    elif layout == "padded_slots":            # head tiles contiguous, heads of a block are not
        shape, strides = (NB, Hkv, bs + 2, D), (Hkv * (bs + 2) * D, (bs + 2) * D, D)
    elif layout == "padded_blocks":           # a block's heads contiguous, blocks spaced out
        shape, strides = (NB, Hkv + 1, bs, D), ((Hkv + 1) * bs * D, bs * D, D)
    else:
        raise ValueError(layout)
    mk = lambda: torch.randint(-32768, 32768, shape, generator=g, device="cuda", dtype=torch.int16).view(torch.bfloat16)
    return mk(), mk(), strides


def shape_of(NB, Hkv, bs, D, strides):
    return binding.Shape(1, Hkv, Hkv, D, bs, NB, 1, *strides)


def u16(t):
    return inputs.as_u16(t).reshape(-1)


CASES = [
    # layout, NB, Hkv, bs, D, n
    ("head_major", 300, 8, 16, 128, 257),      # 32 KiB blocks: two pieces per run
    ("head_major", 200, 8, 32, 128, 131),      # 64 KiB blocks: four pieces
    ("head_major", 64, 2, 16, 64, 40),         # 4 KiB blocks: one short piece
    ("head_major", 5000, 8, 16, 128, 5000),    # more pieces per CTA than the descriptor ring holds
    ("padded_blocks", 90, 8, 16, 128, 77),
    ("padded_slots", 90, 8, 16, 128, 77),      # per-head runs
    ("token_major", 500, 8, 16, 128, 400),     # row by row, many pieces per CTA
    ("head_major", 10, 8, 16, 128, 1),
    ("head_major", 10, 8, 16, 128, 0),
]


@pytest.mark.parametrize("layout,NB,Hkv,bs,D,n", CASES, ids=lambda v: str(v))
def test_gather_scatter_copy_match_oracle(layout, NB, Hkv, bs, D, n):
    k, v, strides = make_pool(layout, NB, Hkv, bs, D, seed=NB + n)
    sh = shape_of(NB, Hkv, bs, D, strides)
    kw = dict(num_kv_heads=Hkv, block_size=bs, head_dim=D, strides=strides)
    cg = torch.Generator().manual_seed(7 + n)
    perm = torch.randperm(NB, generator=cg).to(torch.int32)
    ids = perm[:n].contiguous()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    words = n * Hkv * bs * D

    # gather
    kp = torch.full((max(words, 8),), -1, dtype=torch.int16, device="cuda").view(torch.bfloat16)
    vp = kp.clone()
    binding.kv_gather_blocks(sh, k, v, ids.cuda(), kp, vp, status)
    torch.cuda.synchronize()
    rk, rv = oracle.gather_blocks(u16(k), u16(v), ids.numpy(), **kw)
    assert np.array_equal(u16(kp)[:words], rk.reshape(-1)) and np.array_equal(u16(vp)[:words], rv.reshape(-1))
    assert (u16(kp)[words:] == 0xFFFF).all()

    # scatter the packed blocks into other blocks of a second pool
    k2, v2, _ = make_pool(layout, NB, Hkv, bs, D, seed=1000 + n)
    dst = torch.randperm(NB, generator=cg).to(torch.int32)[:n].contiguous()
    ek, ev = u16(k2).copy(), u16(v2).copy()
    oracle.scatter_blocks(rk, rv, dst.numpy(), ek, ev, **kw)
    binding.kv_scatter_blocks(sh, kp, vp, dst.cuda(), k2, v2, status)
    torch.cuda.synchronize()
    assert np.array_equal(u16(k2), ek) and np.array_equal(u16(v2), ev)       # whole pool, padding included

    # copy inside the first pool: sources and destinations disjoint
    m = min(n, NB // 2)
    src, dstc = perm[:m].contiguous(), perm[NB - m:].contiguous() if m else perm[:0]
    ek, ev = u16(k).copy(), u16(v).copy()
    oracle.copy_blocks(ek, ev, src.numpy(), dstc.numpy(), **kw)
    binding.kv_copy_blocks(sh, k, v, src.cuda(), dstc.cuda(), status)
    torch.cuda.synchronize()
    assert np.array_equal(u16(k), ek) and np.array_equal(u16(v), ev)
    assert int(status.item()) == 0


def test_repeated_sources_and_bad_ids():
    NB, Hkv, bs, D = 50, 8, 16, 128
    k, v, strides = make_pool("head_major", NB, Hkv, bs, D, seed=5)
    sh = shape_of(NB, Hkv, bs, D, strides)
    kw = dict(num_kv_heads=Hkv, block_size=bs, head_dim=D, strides=strides)
    ids = torch.tensor([3, 3, 49, -1, 50, 0, 3, 2**31 - 1], dtype=torch.int32)
    n = ids.numel()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kp = torch.zeros(n * Hkv * bs * D, dtype=torch.bfloat16, device="cuda")
    vp = torch.zeros_like(kp)
    binding.kv_gather_blocks(sh, k, v, ids.cuda(), kp, vp, status)
    torch.cuda.synchronize()
    rk, rv = oracle.gather_blocks(u16(k), u16(v), ids.numpy(), **kw)          # skipped entries stay zero
    assert np.array_equal(u16(kp), rk.reshape(-1)) and np.array_equal(u16(vp), rv.reshape(-1))
    assert int(status.item()) == 4
    ek, ev = u16(k).copy(), u16(v).copy()
    dst = torch.tensor([7, 60, 8, -5, 9, 10, 11, 12], dtype=torch.int32)
    oracle.scatter_blocks(rk, rv, dst.numpy(), ek, ev, **kw)
    binding.kv_scatter_blocks(sh, kp, vp, dst.cuda(), k, v, None)             # status pointer is optional
    torch.cuda.synchronize()
    assert np.array_equal(u16(k), ek) and np.array_equal(u16(v), ev)


def test_migration_of_whole_sequences_keeps_attention_output():
    """Pack the blocks of some sequences, unpack them into fresh blocks of another pool, rewrite the
    block table: decode attention over the migrated sequences is bit-identical."""
    cfg = inputs.DecodeConfig("mig", 32, 8, 128, 16, (inputs.LengthGroup(6, 40, 900),), seed=77, pool_fill=0.6)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    out0 = torch.empty_like(batch.q)
    binding.decode_attention(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, batch.context_lens,
                             cfg.scale, out0, ws)
    lens, table = batch.context_lens.cpu(), batch.block_table.cpu()
    used = [table[b, :(int(lens[b]) + 15) // 16] for b in range(cfg.batch)]
    ids = torch.cat(used).contiguous()
    n = ids.numel()
    kp = torch.empty(n * 8 * 16 * 128, dtype=torch.bfloat16, device="cuda")
    vp = torch.empty_like(kp)
    binding.kv_gather_blocks(sh, batch.k_cache, batch.v_cache, ids.cuda(), kp, vp)
    # receiver: a pool of another size, blocks handed out in another order
    NB2 = n + 13
    k2 = torch.full((NB2, 8, 16, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    v2 = torch.full_like(k2, float("nan"))
    new_ids = torch.randperm(NB2, generator=torch.Generator().manual_seed(3)).to(torch.int32)[:n].contiguous()
    sh2 = binding.Shape(sh.batch, sh.num_q_heads, sh.num_kv_heads, sh.head_dim, sh.block_size, NB2,
                        sh.max_blocks_per_seq, sh.kv_block_stride, sh.kv_head_stride, sh.kv_token_stride)
    binding.kv_scatter_blocks(sh2, kp, vp, new_ids.cuda(), k2, v2)
    table2 = torch.full_like(table, -1)
    off = 0
    for b, u in enumerate(used):
        table2[b, :u.numel()] = new_ids[off:off + u.numel()]
        off += u.numel()
    out1 = torch.empty_like(batch.q)
    ws2 = torch.empty(binding.workspace_bytes(sh2), dtype=torch.uint8, device="cuda")
    binding.decode_attention(sh2, batch.q, k2, v2, table2.cuda(), batch.context_lens, cfg.scale, out1, ws2)
    torch.cuda.synchronize()
    assert torch.equal(out0.view(torch.int16), out1.view(torch.int16))
