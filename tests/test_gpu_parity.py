"""CUDA path vs the fp64 CPU oracle, through the C ABI (needs a B200)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs
from util import assert_parity, gpu_attention, oracle_attention

pytestmark = pytest.mark.gpu
G = inputs.LengthGroup
C = inputs.DecodeConfig


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


DEFAULT_KNOBS = dict(warps=4, stages=0, ctas_per_sm=2, chunk_min=256, chunk_max=8192, items_per_cta=6, split_halves=0,
                     tiles_per_warp=1, pdl=1)


def fixed(*vals):
    return (G(len(vals), min(vals), max(vals), "fixed", tuple(vals)),)


SMALL = [
    inputs.CONFIGS["cfg0"],
    dataclasses.replace(inputs.CONFIGS["cfg0"], layout="token_major", seed=30, name="cfg0-token-major"),
    # every tail length around tile / stage / block boundaries, and an empty sequence
    C("edges-d64", 8, 2, 64, 16, fixed(0, 1, 2, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 257), seed=31,
      shuffle_batch=False),
    C("edges-d128", 32, 8, 128, 16, fixed(1, 16, 17, 48, 63, 64, 65, 100, 191, 192, 193, 300), seed=32, pool_fill=0.7),
    C("g1-mha", 4, 4, 128, 16, (G(6, 1, 400),), seed=33),
    C("g5-bs32", 40, 8, 128, 32, (G(6, 1, 700),), seed=34, pool_fill=0.8),
    C("g8-bs32", 64, 8, 128, 32, (G(5, 1, 900),), seed=35, sigma=0.5),
    C("g16", 32, 2, 128, 16, (G(4, 1, 500),), seed=36),
    C("g12-d64", 24, 2, 64, 32, (G(4, 1, 500),), seed=37),
    C("bs64", 16, 4, 128, 64, (G(5, 1, 600),), seed=38),
    C("bs128", 16, 4, 128, 128, (G(5, 1, 900),), seed=39),
    C("bs256-d64", 8, 2, 64, 256, (G(4, 1, 1200),), seed=40),
    C("token-major-d128", 32, 8, 128, 16, (G(6, 1, 500),), seed=41, layout="token_major", pool_fill=0.75),
    # long enough to be split into several chunks (several stages, ragged last chunk)
    C("split", 32, 8, 128, 16, fixed(5000, 37, 2049, 1025, 300, 9999), seed=42, pool_fill=0.9, shuffle_batch=False),
    C("split-g8-bs32", 64, 8, 128, 32, fixed(20000, 129, 4097, 64), seed=43, sigma=0.5, shuffle_batch=False),
    # more sequences than the plan keeps in shared memory (its global-memory path), many of them empty or tiny
    C("batch-5000", 8, 2, 128, 16, (G(5000, 0, 40),), seed=44, pool_fill=0.9),
    C("batch-4200-d64", 8, 2, 64, 16, (G(4200, 0, 70),), seed=45),
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_attention_matches_oracle(cfg):
    batch = inputs.make_batch(cfg, "cuda", poison=True, table_pad=2**31 - 1)
    out = gpu_attention(batch)
    ref = oracle_attention(batch)
    assert_parity(out, ref.out, what=cfg.name)
    for b in range(cfg.batch):
        if int(batch.context_lens[b]) == 0:
            assert torch.count_nonzero(out[b].float()) == 0


@pytest.mark.parametrize("knobs", [dict(warps=2), dict(warps=8, ctas_per_sm=1), dict(warps=4, ctas_per_sm=1),
                                   dict(warps=2, ctas_per_sm=3), dict(split_halves=1), dict(stages=2),
                                   dict(chunk_min=128, chunk_max=128), dict(tiles_per_warp=2),
                                   dict(tiles_per_warp=2, warps=2, ctas_per_sm=3), dict(pdl=0)],
                         ids=lambda k: "-".join(f"{a}{b}" for a, b in k.items()))
def test_launch_shapes_agree_with_oracle(knobs):
    default = dict(DEFAULT_KNOBS)
    try:
        binding.set_tuning(**{**default, **knobs})
        for cfg in (SMALL[3], SMALL[5], SMALL[13], SMALL[2], SMALL[7], SMALL[10]):
            batch = inputs.make_batch(cfg, "cuda", poison=True, table_pad=-1)
            assert_parity(gpu_attention(batch), oracle_attention(batch).out, what=f"{cfg.name} {knobs}")
    finally:
        binding.set_tuning(**default)


def test_context_one_returns_value_bit_exact():
    cfg = C("one", 32, 8, 128, 16, fixed(1, 1, 1, 1), seed=44)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    out = gpu_attention(batch)
    for b in range(4):
        blk = int(batch.block_table[b, 0])
        want = batch.v_cache[blk, :, 0, :].repeat_interleave(4, dim=0)      # [Hq, D]
        assert torch.equal(out[b].view(torch.int16), want.view(torch.int16))


def test_identical_keys_give_mean_of_values():
    cfg = C("mean", 32, 8, 128, 16, fixed(64, 200), seed=45)
    batch = inputs.make_batch(cfg, "cuda", poison=False)
    batch.k_cache[:] = batch.k_cache[0, :, 0, :].clone().view(1, 8, 1, 128)
    out = gpu_attention(batch)
    ref = oracle_attention(batch)
    assert_parity(out, ref.out, what="mean")


def test_block_permutation_and_rerun_are_bit_identical():
    cfg = SMALL[13]
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    out1 = gpu_attention(batch)
    out2 = gpu_attention(batch)
    assert torch.equal(out1.view(torch.int16), out2.view(torch.int16))        # run-to-run determinism
    g = torch.Generator().manual_seed(5)
    perm = torch.randperm(batch.num_blocks, generator=g).cuda()
    k2, v2 = torch.empty_like(batch.k_cache), torch.empty_like(batch.v_cache)
    k2[perm], v2[perm] = batch.k_cache, batch.v_cache
    t2 = batch.block_table.clone()
    ok = t2 >= 0
    t2[ok] = perm[t2[ok].long()].to(torch.int32)
    moved = dataclasses.replace(batch, k_cache=k2, v_cache=v2, block_table=t2)
    out3 = gpu_attention(moved)
    assert torch.equal(out1.view(torch.int16), out3.view(torch.int16))        # block indexing is exact


def test_shared_prefix_blocks_are_legal():
    cfg = C("shared", 32, 8, 128, 16, fixed(160, 160), seed=46)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    batch.block_table[1, :5] = batch.block_table[0, :5]                        # both read the same 80 tokens
    assert_parity(gpu_attention(batch), oracle_attention(batch).out, what="shared prefix")


def test_out_of_pool_table_entry_reads_zeros_and_does_not_fault():
    cfg = C("oob", 8, 2, 128, 16, fixed(48), seed=47)
    batch = inputs.make_batch(cfg, "cuda", poison=False)
    batch.block_table[0, 1] = batch.num_blocks + 7
    out = gpu_attention(batch)
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_kv_append_bit_exact(layout):
    cfg = C("append", 32, 8, 128, 16, (G(37, 1, 300),), seed=48, pool_fill=0.8, layout=layout)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    lens = batch.context_lens.clone()
    lens[0], lens[1] = 32, 15                                                   # block boundary / last slot
    batch = inputs.make_batch(cfg, "cuda", poison=True, context_lens=lens)
    k_ref, v_ref = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    n = oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k_ref, v_ref,
                         batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(),
                         block_size=16, strides=batch.strides)
    assert n == 37
    binding.kv_append(binding.shape_of(batch), batch.k_new, batch.v_new, batch.k_cache, batch.v_cache,
                      batch.block_table, batch.context_lens)
    torch.cuda.synchronize()
    assert np.array_equal(inputs.as_u16(batch.k_cache), k_ref)                 # whole pool, word for word
    assert np.array_equal(inputs.as_u16(batch.v_cache), v_ref)


def test_kv_append_skips_bad_positions():
    cfg = C("append-skip", 8, 2, 64, 16, fixed(5, 20, 33), seed=49)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    pos = torch.tensor([-1, batch.max_blocks_per_seq * 16, 33], dtype=torch.int32, device="cuda")
    k_ref, v_ref = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k_ref, v_ref,
                     batch.block_table.cpu().numpy(), pos.cpu().numpy(), block_size=16, strides=batch.strides)
    binding.kv_append(binding.shape_of(batch), batch.k_new, batch.v_new, batch.k_cache, batch.v_cache,
                      batch.block_table, pos)
    torch.cuda.synchronize()
    assert np.array_equal(inputs.as_u16(batch.k_cache), k_ref) and np.array_equal(inputs.as_u16(batch.v_cache), v_ref)


@pytest.mark.parametrize("pinned,stage_knob,hq", [(True, 1, 32), (True, 2, 32), (True, 1, 128), (False, 1, 32)],
                         ids=["page-locked", "page-locked-q-staged", "page-locked-16-heads-per-kv-head", "pageable"])
def test_serving_step_from_host_buffers(pinned, stage_knob, hq):
    """append at T then attend T + 1 through the host-buffer entry point: page-locked buffers are read
    through their device mapping (q by the attention kernel itself, or staged by the first launch: behind
    the knob and for the 16-row kernel) and the result is written to the host directly; pageable ones are
    copied."""
    launches = 3
    cfg = C("step", hq, 8, 128, 16, (G(9, 1, 2500),), seed=50, pool_fill=0.8)
    binding.set_tuning(host_stage_kernel=stage_knob)
    try:
        _serving_step_from_host_buffers(cfg, pinned, launches)
    finally:
        binding.set_tuning(host_stage_kernel=1)


def _serving_step_from_host_buffers(cfg, pinned, launches):
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    pin = (lambda t: t.cpu().contiguous().pin_memory()) if pinned else (lambda t: t.cpu().contiguous().clone())
    pos = pin(batch.context_lens)
    lens1 = pin(batch.context_lens + 1)
    out_h = torch.full(batch.q.shape, float("nan"), dtype=torch.bfloat16)
    out_h = out_h.pin_memory() if pinned else out_h
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    stg = torch.empty(binding.step_staging_bytes(sh), dtype=torch.uint8, device="cuda")
    k_ref, v_ref = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    binding.decode_step_host(sh, pin(batch.q), pin(batch.k_new), pin(batch.v_new), pin(batch.block_table), pos, lens1,
                             batch.k_cache, batch.v_cache, cfg.scale, out_h, stg, ws)
    assert binding.workspace_status(ws) == 0
    oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k_ref, v_ref,
                     batch.block_table.cpu().numpy(), pos.numpy(), block_size=16, strides=batch.strides)
    assert np.array_equal(inputs.as_u16(batch.k_cache), k_ref)
    ref = oracle.decode_attention(inputs.as_u16(batch.q), k_ref, v_ref, batch.block_table.cpu().numpy(),
                                  lens1.numpy(), cfg.scale, num_kv_heads=8, block_size=16, strides=batch.strides)
    assert_parity(out_h, ref.out, what="host step")
    assert binding.last_launch_count() == launches


def test_refused_fused_step_enqueues_nothing():
    """A call that returns an argument error has touched no buffer: the fused step with a workspace that is too
    small (or misaligned) leaves the pool, `out` and the workspace as they were."""
    cfg = C("refused", 32, 8, 128, 16, (G(6, 100, 900),), seed=53)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    ws = torch.zeros(binding.workspace_bytes(sh) + 256, dtype=torch.uint8, device="cuda")
    out = torch.full_like(batch.q, float("nan"))
    lens1 = (batch.context_lens + 1).contiguous()
    k0, v0 = batch.k_cache.clone(), batch.v_cache.clone()
    for bad_ws in (ws[:1024], ws[16:]):                                        # too small; not 256-byte aligned
        with pytest.raises(binding.OocoError) as err:
            binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                                batch.context_lens, lens1, cfg.scale, out, bad_ws)
        assert err.value.status == -4
    with pytest.raises(binding.OocoError) as err:                              # softmax scale must be positive
        binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                            batch.context_lens, lens1, 0.0, out, ws[:binding.workspace_bytes(sh)])
    assert err.value.status == -2
    torch.cuda.synchronize()
    assert torch.equal(batch.k_cache.view(torch.int16), k0.view(torch.int16))
    assert torch.equal(batch.v_cache.view(torch.int16), v0.view(torch.int16))
    assert torch.isnan(out.float()).all() and int(ws.count_nonzero()) == 0


def test_fused_step_on_device_buffers():
    """ooco_decode_step = append at T (bit-exact over the whole pool) + attention over T + 1 tokens."""
    cfg = C("fused", 40, 8, 128, 16, (G(21, 1, 3000),), seed=52, pool_fill=0.85)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    out = torch.full_like(batch.q, float("nan"))
    lens1 = (batch.context_lens + 1).contiguous()
    k_ref, v_ref = inputs.as_u16(batch.k_cache).copy(), inputs.as_u16(batch.v_cache).copy()
    for _ in range(2):                                                         # same slots twice: idempotent
        binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                            batch.context_lens, lens1, cfg.scale, out, ws)
    assert binding.workspace_status(ws) == 0
    oracle.kv_append(inputs.as_u16(batch.k_new), inputs.as_u16(batch.v_new), k_ref, v_ref,
                     batch.block_table.cpu().numpy(), batch.context_lens.cpu().numpy(), block_size=16,
                     strides=batch.strides)
    assert np.array_equal(inputs.as_u16(batch.k_cache), k_ref) and np.array_equal(inputs.as_u16(batch.v_cache), v_ref)
    ref = oracle.decode_attention(inputs.as_u16(batch.q), k_ref, v_ref, batch.block_table.cpu().numpy(),
                                  lens1.cpu().numpy(), cfg.scale, num_kv_heads=8, block_size=16, strides=batch.strides)
    assert_parity(out, ref.out, what="fused step")


def test_many_sequences_plan_scan():
    """More sequences than plan threads: exercises the multi-pass scan of the plan kernel."""
    cfg = C("many", 8, 2, 64, 16, (G(2500, 0, 40), G(3, 600, 900)), seed=51)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    assert_parity(gpu_attention(batch), oracle_attention(batch).out, what="many")


def test_step_replays_from_a_cuda_graph():
    """The three launches of ooco_decode_step (programmatic dependent launches included) are captured
    into a CUDA graph once and replayed: same bits as the direct call, also after the inputs change."""
    cfg = C("graph", 32, 8, 128, 16, (G(12, 1, 3000),), seed=55, pool_fill=0.9)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
    lens1 = (batch.context_lens + 1).contiguous()
    out_direct, out_graph = torch.empty_like(batch.q), torch.full_like(batch.q, float("nan"))
    binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                        batch.context_lens, lens1, cfg.scale, out_direct, ws)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                            batch.context_lens, lens1, cfg.scale, out_graph, ws, side)
        graph.capture_end()
    graph.replay()
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    assert torch.equal(out_direct.view(torch.int16), out_graph.view(torch.int16))
    # new query values in the same buffers: the replay picks them up
    batch.q.copy_(torch.randn_like(batch.q.float()).to(torch.bfloat16))
    binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, batch.k_cache, batch.v_cache, batch.block_table,
                        batch.context_lens, lens1, cfg.scale, out_direct, ws)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out_direct.view(torch.int16), out_graph.view(torch.int16))
    ref = oracle_attention(batch, context_lens=lens1)
    assert_parity(out_graph, ref.out, what="graph replay")


def test_kv_head_sharding_needs_no_exchange():
    """Tensor-parallel layout: each of two ranks holds half of the kv heads of the pool and the
    matching query heads; their outputs, side by side on the head axis, are the unsharded result."""
    cfg = C("tp2", 32, 8, 128, 16, (G(9, 1, 2500),), seed=57, pool_fill=0.8)
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    ref = oracle_attention(batch)
    outs = []
    for rank in range(2):
        k = batch.k_cache[:, 4 * rank:4 * rank + 4].contiguous()             # [NB, Hkv / 2, bs, D]
        v = batch.v_cache[:, 4 * rank:4 * rank + 4].contiguous()
        q = batch.q[:, 16 * rank:16 * rank + 16].contiguous()
        sh = binding.Shape(cfg.batch, 16, 4, 128, 16, batch.num_blocks, batch.max_blocks_per_seq, 4 * 16 * 128, 16 * 128, 128)
        ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device="cuda")
        out = torch.full_like(q, float("nan"))
        binding.decode_attention(sh, q, k, v, batch.block_table, batch.context_lens, cfg.scale, out, ws)
        assert binding.workspace_status(ws) == 0
        outs.append(out)
    assert_parity(torch.cat(outs, dim=1), ref.out, what="kv-head sharding")
