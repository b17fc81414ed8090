"""Helpers shared by the parity tests: run the CUDA path, run the oracle, compare."""
import numpy as np
import torch

import oracle
from paper_2511_21862_b200 import binding, inputs

MAX_ABS_TOL = 1e-2    # bf16 in / fp32 accumulate / bf16 out vs the fp64 oracle: max |err|
MEAN_ABS_TOL = 1e-3   # and mean |err|, over all B * Hq * D outputs


import contextlib


@contextlib.contextmanager
def fp32_output():
    """The library's diagnostic output mode: `out` tensors are fp32 and hold the values before the bf16 rounding."""
    binding.set_tuning(out_f32=1)
    try:
        yield
    finally:
        binding.set_tuning(out_f32=0)


def assert_parity_and_rounding(out_bf16: torch.Tensor, out_f32: torch.Tensor, ref: np.ndarray, what=""):
    """The stated tolerance on the fp32 output (no allowance for the output format), and the bf16 output must be
    exactly the fp32 output rounded to nearest even: together they hold the bf16 path to the same arithmetic."""
    mx, mean = assert_parity(out_f32, ref, what=what + " (fp32 out)")
    want = out_f32.to(torch.bfloat16)
    assert torch.equal(out_bf16.view(torch.int16), want.view(torch.int16)), f"{what}: bf16 out is not round(fp32 out)"
    return mx, mean


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def gpu_attention(batch, context_lens=None, scale=None, check_status=True):
    """out (bf16, device) of ooco_decode_attention on a device-resident batch."""
    sh = binding.shape_of(batch)
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device=batch.q.device)
    out = torch.full_like(batch.q, float("nan"))
    lens = batch.context_lens if context_lens is None else context_lens
    binding.decode_attention(sh, batch.q, batch.k_cache, batch.v_cache, batch.block_table, lens,
                             batch.cfg.scale if scale is None else scale, out, ws)
    if check_status:
        assert binding.workspace_status(ws) == 0
    torch.cuda.synchronize()
    return out


def oracle_attention(batch, context_lens=None, scale=None, seqs=None, kv8=None):
    """fp64 oracle on a host copy; with `seqs`, only those sequences (other rows NaN), using a
    compacted copy of just their blocks (plain torch indexing) so huge pools need not be copied.
    `kv8` = (k_scale, v_scale): the pools hold E4M3 codes (the 8-bit oracle)."""
    cfg = batch.cfg
    lens = (batch.context_lens if context_lens is None else context_lens).cpu()
    table = batch.block_table.cpu()
    k, v = batch.k_cache, batch.v_cache
    pairs = None
    if seqs is not None:
        seqs = [int(s) for s in seqs]
        bs = cfg.block_size
        new_table = table.clone()
        ids = []
        for b in seqs:
            n = (int(lens[b]) + bs - 1) // bs
            new_table[b, :n] = torch.arange(len(ids), len(ids) + n, dtype=torch.int32)
            ids.extend(table[b, :n].tolist())
        idx = torch.tensor(ids if ids else [0], dtype=torch.long, device=k.device)
        k, v, table = k.index_select(0, idx), v.index_select(0, idx), new_table
        pairs = np.array([(b, h) for b in seqs for h in range(cfg.num_q_heads)], dtype=np.int32)
    if kv8 is not None:
        return oracle.decode_attention_fp8(
            inputs.as_u16(batch.q), inputs.as_u8(k), inputs.as_u8(v), table.numpy(), lens.numpy(),
            cfg.scale if scale is None else scale, kv8[0], kv8[1], num_kv_heads=cfg.num_kv_heads,
            block_size=cfg.block_size, strides=batch.strides, pairs=pairs)
    return oracle.decode_attention(
        inputs.as_u16(batch.q), inputs.as_u16(k), inputs.as_u16(v), table.numpy(), lens.numpy(),
        cfg.scale if scale is None else scale, num_kv_heads=cfg.num_kv_heads, block_size=cfg.block_size,
        strides=batch.strides, pairs=pairs)


def sequence_slices(lens, block_size, block_bytes, slice_bytes):
    """Consecutive runs of sequences whose cache blocks add up to at most `slice_bytes` each
    (a single sequence larger than that is a run of its own)."""
    runs, cur, acc = [], [], 0
    for b, T in enumerate(int(x) for x in lens):
        need = -(-T // block_size) * block_bytes
        if cur and acc + need > slice_bytes:
            runs.append(cur)
            cur, acc = [], 0
        cur.append(b)
        acc += need
    if cur:
        runs.append(cur)
    return runs


def oracle_attention_every_sequence(batch, context_lens=None, scale=None, kv8=None, slice_bytes=3 << 30):
    """The oracle's output for EVERY sequence of a batch whose pool is too large to copy to the host in
    one piece: the sequences are taken in consecutive runs, each run gets a compacted host copy of just
    its blocks, and the rows are put together.  fp64 [B, Hq, D]."""
    cfg = batch.cfg
    lens = (batch.context_lens if context_lens is None else context_lens).cpu()
    block_bytes = 2 * cfg.num_kv_heads * cfg.block_size * cfg.head_dim * batch.k_cache.element_size()
    out = np.full(tuple(batch.q.shape), np.nan, dtype=np.float64)
    for run in sequence_slices(lens.tolist(), cfg.block_size, block_bytes, slice_bytes):
        r = oracle_attention(batch, context_lens=lens, scale=scale, seqs=run, kv8=kv8)
        out[run] = r.out[run]
    assert not np.isnan(out).any()
    return out


def assert_parity(out_gpu: torch.Tensor, ref: np.ndarray, rows=None, what=""):
    got = bf16_to_f64(out_gpu)
    if rows is not None:
        got, ref = got[rows], ref[rows]
    assert not np.isnan(ref).any(), "oracle rows missing"
    assert not np.isnan(got).any(), f"{what}: NaN in the CUDA output"
    err = np.abs(got - ref)
    assert err.max() <= MAX_ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert err.mean() <= MEAN_ABS_TOL, f"{what}: mean abs err {err.mean():.3e}"
    return float(err.max()), float(err.mean())
