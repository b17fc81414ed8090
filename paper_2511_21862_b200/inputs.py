"""Seeded synthetic decode batches (inputs only; none of the operator's arithmetic lives here).

The batches stand in for the paper's request traces: a decode batch holds every online
request plus the offline requests the scheduler admitted, in random order (Algorithm
"Mix Decoding Selection"), so a batch is a mix of short and long contexts over a paged,
non-contiguous KV pool.  Both the CUDA path and the CPU oracle are fed from here.

Lengths and block tables are always drawn on the CPU generator (identical on every
machine); the large value tensors (q, pool, new K/V) are drawn on the target device.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace

import torch


@dataclass(frozen=True)
class LengthGroup:
    """`count` sequences with context lengths drawn from [lo, hi] (inclusive)."""
    count: int
    lo: int
    hi: int
    dist: str = "uniform"          # "uniform" | "loguniform" | "fixed" (uses `values`)
    values: tuple = ()


@dataclass(frozen=True)
class DecodeConfig:
    name: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    groups: tuple                   # tuple[LengthGroup, ...]
    seed: int
    sigma: float = 1.0              # std of q / k / v values
    pool_fill: float = 1.0          # used blocks / pool blocks
    pool_blocks: int = 0            # explicit pool size (0: derive from pool_fill)
    shuffle_batch: bool = True      # random order of online / offline sequences in the batch
    layout: str = "head_major"      # "head_major" [NB,Hkv,bs,D] | "token_major" [NB,bs,Hkv,D]
    description: str = ""

    @property
    def batch(self) -> int:
        return sum(g.count for g in self.groups)

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)


# The five benchmark workloads.
CONFIGS = {
    "cfg0": DecodeConfig(
        "cfg0", 8, 2, 64, 16, (LengthGroup(4, 17, 256, "fixed", (17, 64, 130, 256)),), seed=0,
        pool_blocks=64, shuffle_batch=False,
        description="tiny: B 4, 8q/2kv heads, D 64, block 16, contexts {17,64,130,256}, 64-block pool"),
    "cfg1": DecodeConfig(
        "cfg1", 32, 8, 128, 16, (LengthGroup(48, 256, 2048), LengthGroup(16, 2048, 8192)), seed=1,
        description="Llama-3-8B shape: B 64 = 48 online U[256,2048] + 16 offline U[2048,8192]"),
    "cfg2": DecodeConfig(
        "cfg2", 40, 8, 128, 16,
        (LengthGroup(32, 512, 4096), LengthGroup(224, 4096, 32768, "loguniform")), seed=2,
        description="Qwen2.5-32B shape: B 256 = 32 online U[512,4096] + 224 offline logU[4096,32768]"),
    "cfg3": DecodeConfig(
        "cfg3", 64, 8, 128, 32, (LengthGroup(115, 128, 1024), LengthGroup(13, 32768, 65536)), seed=3,
        sigma=0.5,
        description="Llama-3-70B shape: B 128, 90% U[128,1024] + 10% U[32768,65536], block 32, sigma 0.5"),
    "cfg4": DecodeConfig(
        "cfg4", 32, 8, 128, 16, (LengthGroup(512, 1024, 16384),), seed=4, pool_fill=0.9,
        description="fragmentation: Llama-3-8B shape, B 512 U[1024,16384], 90%-full pool, then append"),
}


def scaled_config(cfg: DecodeConfig, *, batch_div: int = 1, len_div: int = 1, name: str | None = None):
    """A smaller sibling of `cfg` (fewer sequences, shorter contexts) with the same structure."""
    groups = []
    for g in cfg.groups:
        cnt = max(1, g.count // batch_div)
        if g.dist == "fixed":
            groups.append(replace(g, count=min(cnt, len(g.values)), values=g.values[:cnt]))
        else:
            groups.append(replace(g, count=cnt, lo=max(1, g.lo // len_div), hi=max(2, g.hi // len_div)))
    return replace(cfg, groups=tuple(groups), name=name or f"{cfg.name}/b{batch_div}/l{len_div}")


def draw_context_lens(cfg: DecodeConfig, gen: torch.Generator) -> torch.Tensor:
    """int32 [B] context lengths, groups concatenated then (optionally) shuffled."""
    parts = []
    for g in cfg.groups:
        if g.dist == "fixed":
            parts.append(torch.tensor(g.values[: g.count], dtype=torch.int64))
        elif g.dist == "uniform":
            parts.append(torch.randint(g.lo, g.hi + 1, (g.count,), generator=gen, dtype=torch.int64))
        elif g.dist == "loguniform":
            u = torch.rand((g.count,), generator=gen, dtype=torch.float64)
            x = torch.exp(math.log(g.lo) + u * (math.log(g.hi) - math.log(g.lo)))
            parts.append(x.round().to(torch.int64).clamp_(g.lo, g.hi))
        else:
            raise ValueError(g.dist)
    lens = torch.cat(parts)
    if cfg.shuffle_batch:
        lens = lens[torch.randperm(lens.numel(), generator=gen)]
    return lens.to(torch.int32)


@dataclass
class DecodeBatch:
    cfg: DecodeConfig
    q: torch.Tensor              # bf16 [B, Hq, D]
    k_cache: torch.Tensor        # bf16 pool, [NB, Hkv, bs, D] or [NB, bs, Hkv, D]
    v_cache: torch.Tensor
    block_table: torch.Tensor    # int32 [B, MB]
    context_lens: torch.Tensor   # int32 [B]
    k_new: torch.Tensor          # bf16 [B, Hkv, D]  (token to append at position context_lens[b])
    v_new: torch.Tensor
    num_blocks: int
    strides: tuple               # (block, head, token) element strides of the pool
    extras: dict = field(default_factory=dict)

    @property
    def max_blocks_per_seq(self) -> int:
        return self.block_table.shape[1]

    @property
    def total_tokens(self) -> int:
        return int(self.context_lens.to(torch.int64).sum())


def _randn_bf16(shape, sigma, gen, device, chunk_elems=1 << 28):
    """bf16 = round-to-nearest of fp32 normals, drawn in bounded chunks along dim 0."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        x = torch.randn(e - s, generator=gen, device=device, dtype=torch.float32)
        if sigma != 1.0:
            x.mul_(sigma)
        flat[s:e] = x.to(torch.bfloat16)
    return out


@dataclass
class BatchLayout:
    """Everything of a batch that is drawn on the CPU generator: lengths, block table, pool size."""
    lens: torch.Tensor           # int32 [B]
    table: torch.Tensor          # int32 [B, MB]
    nblk: torch.Tensor           # int64 [B] blocks owned by each sequence (room for the append included)
    num_blocks: int              # NB
    used_blocks: int
    valid_slots: torch.Tensor    # int32 [NB] tokens < T_b held by each block


def draw_layout(cfg: DecodeConfig, *, table_pad: int = -1, context_lens: torch.Tensor | None = None) -> BatchLayout:
    """Lengths and block table of `cfg` (identical on every machine: CPU generator, seed of the config)."""
    cgen = torch.Generator(device="cpu").manual_seed(cfg.seed)
    lens = draw_context_lens(cfg, cgen) if context_lens is None else context_lens.to(torch.int32).cpu()
    B, bs = lens.numel(), cfg.block_size
    nblk = (lens.to(torch.int64) + 1 + bs - 1) // bs           # blocks owned, incl. room for the append
    used = int(nblk.sum())
    if cfg.pool_blocks:
        NB = cfg.pool_blocks
    else:
        NB = int(math.ceil(used / cfg.pool_fill))
    assert NB >= used, (NB, used)
    MB = int(nblk.max())
    perm = torch.randperm(NB, generator=cgen)[:used].to(torch.int32)
    table = torch.full((B, MB), table_pad, dtype=torch.int32)
    valid_slots = torch.zeros(NB, dtype=torch.int32)             # tokens < T_b held by each block
    off = 0
    for b in range(B):
        n = int(nblk[b])
        ids = perm[off:off + n]
        table[b, :n] = ids
        T = int(lens[b])
        cnt = torch.clamp(T - torch.arange(n, dtype=torch.int64) * bs, 0, bs).to(torch.int32)
        valid_slots[ids.long()] = cnt
        off += n
    return BatchLayout(lens, table, nblk, NB, used, valid_slots)


def make_batch(cfg: DecodeConfig, device="cpu", *, poison: bool = True, table_pad: int = -1,
               context_lens: torch.Tensor | None = None) -> DecodeBatch:
    """Draw one decode batch.

    Every sequence owns ceil((T_b + 1) / bs) distinct physical blocks (room for the one-token
    append at position T_b), taken from a random permutation of the pool, so tables are shuffled
    and non-contiguous; with pool_fill < 1 the unused blocks are holes spread over the pool.
    With `poison`, every slot at or beyond T_b (and every unused block) is NaN and every table
    entry beyond a sequence's blocks is `table_pad`, so any out-of-range read shows up.
    """
    device = torch.device(device)
    lay = draw_layout(cfg, table_pad=table_pad, context_lens=context_lens)
    lens, table, NB, used, valid_slots = lay.lens, lay.table, lay.num_blocks, lay.used_blocks, lay.valid_slots
    B, bs, Hkv, Hq, D = lens.numel(), cfg.block_size, cfg.num_kv_heads, cfg.num_q_heads, cfg.head_dim

    dgen = torch.Generator(device=device).manual_seed(cfg.seed + 1000)
    if cfg.layout == "head_major":
        pshape, strides = (NB, Hkv, bs, D), (Hkv * bs * D, bs * D, D)
        slot_dim = 2
    elif cfg.layout == "token_major":
        pshape, strides = (NB, bs, Hkv, D), (bs * Hkv * D, D, Hkv * D)
        slot_dim = 1
    else:
        raise ValueError(cfg.layout)
    k_cache = _randn_bf16(pshape, cfg.sigma, dgen, device)
    v_cache = _randn_bf16(pshape, cfg.sigma, dgen, device)
    q = _randn_bf16((B, Hq, D), cfg.sigma, dgen, device)
    k_new = _randn_bf16((B, Hkv, D), cfg.sigma, dgen, device)
    v_new = _randn_bf16((B, Hkv, D), cfg.sigma, dgen, device)
    if poison:
        vs = valid_slots.to(device)
        slot = torch.arange(bs, device=device, dtype=torch.int32)
        view = [1, 1, 1, 1]
        view[slot_dim] = bs
        step = max(1, (1 << 26) // (Hkv * bs * D))               # blocks per masking chunk
        for s in range(0, NB, step):
            e = min(NB, s + step)
            dead = slot.view(view) >= vs[s:e].view(-1, 1, 1, 1)  # [nb,1,bs,1] or [nb,bs,1,1]
            k_cache[s:e].masked_fill_(dead, float("nan"))
            v_cache[s:e].masked_fill_(dead, float("nan"))
    return DecodeBatch(cfg, q, k_cache, v_cache, table.to(device), lens.to(device), k_new, v_new,
                       NB, strides, extras={"used_blocks": used, "valid_slots": valid_slots})


def make_sample_batch(cfg: DecodeConfig, seqs, device="cpu") -> DecodeBatch:
    """The sequences `seqs` of `cfg`'s batch alone, over a pool that holds just their blocks.

    Lengths and block-table rows are those of the full batch (same CPU draws); the sampled sequences'
    blocks are renumbered in the shuffled order of their original ids, so the compact pool is as
    non-contiguous as the original one.  Values are drawn for the sampled blocks only (same
    distribution as `make_batch`, other draws), which keeps the host footprint to the sample's size.
    The batch index of sequence seqs[i] is i."""
    device = torch.device(device)
    lay = draw_layout(cfg)
    seqs = [int(b) for b in seqs]
    bs, Hkv, Hq, D = cfg.block_size, cfg.num_kv_heads, cfg.num_q_heads, cfg.head_dim
    ids = torch.cat([lay.table[b, : int(lay.nblk[b])] for b in seqs]).to(torch.int64)
    order = torch.argsort(ids)                                   # rank of each original id = its new id
    new_id = torch.empty_like(order)
    new_id[order] = torch.arange(ids.numel())
    NB, MB = ids.numel(), int(max(int(lay.nblk[b]) for b in seqs))
    table = torch.full((len(seqs), MB), -1, dtype=torch.int32)
    off = 0
    for i, b in enumerate(seqs):
        n = int(lay.nblk[b])
        table[i, :n] = new_id[off:off + n].to(torch.int32)
        off += n
    lens = lay.lens[seqs].contiguous()
    dgen = torch.Generator(device=device).manual_seed(cfg.seed + 2000)
    assert cfg.layout == "head_major"
    k_cache = _randn_bf16((NB, Hkv, bs, D), cfg.sigma, dgen, device)
    v_cache = _randn_bf16((NB, Hkv, bs, D), cfg.sigma, dgen, device)
    q = _randn_bf16((len(seqs), Hq, D), cfg.sigma, dgen, device)
    k_new = _randn_bf16((len(seqs), Hkv, D), cfg.sigma, dgen, device)
    v_new = _randn_bf16((len(seqs), Hkv, D), cfg.sigma, dgen, device)
    return DecodeBatch(cfg, q, k_cache, v_cache, table.to(device), lens.to(device), k_new, v_new, NB,
                       (Hkv * bs * D, bs * D, D), extras={"used_blocks": NB, "sampled_from": seqs})


def as_u16(t: torch.Tensor):
    """Raw bit patterns of a bf16 tensor as a numpy uint16 array (host copy)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")


def to_e4m3_pool(batch: DecodeBatch, k_scale: float, v_scale: float, *, poison: bool = True) -> DecodeBatch:
    """The same batch with 8-bit (E4M3) caches: code = nearest E4M3 of value / scale, made with the
    library dtype cast (this only synthesises stored data; both the CUDA path and the oracle read the
    codes).  Values beyond the format's range are clamped first.  With `poison`, every slot that held
    NaN (slots at or beyond T_b, unused blocks) holds the NaN code."""
    def conv(x, s):
        out = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
        step = max(1, (1 << 26) // max(1, x[0].numel()))
        for a in range(0, x.shape[0], step):
            y = x[a:a + step].float() / s
            nan = torch.isnan(y)
            c = y.clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
            out[a:a + step] = torch.where(nan, torch.full_like(c, 0x7F if poison else 0), c)
        return out
    return replace(batch, k_cache=conv(batch.k_cache, k_scale), v_cache=conv(batch.v_cache, v_scale),
                   extras=dict(batch.extras, k_scale=float(k_scale), v_scale=float(v_scale)))


def as_u8(t: torch.Tensor):
    """Host numpy uint8 copy of a uint8 tensor."""
    return t.detach().cpu().contiguous().numpy()
