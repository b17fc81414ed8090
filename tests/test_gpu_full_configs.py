"""Full-size workloads (the benchmark's configurations and launch shape) vs the oracle.

cfg1 is compared on every output.  For the larger pools the oracle is run on a sample of whole
sequences (the longest, the shortest and a few in between; all their q heads), from a host copy of
just those sequences' blocks; the append of the fragmentation workload is compared word for word
over the entire pool.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21862_b200 import binding, build, inputs
from util import assert_parity, gpu_attention, oracle_attention

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def sample_sequences(lens: torch.Tensor, n_each=3):
    order = torch.argsort(lens.cpu())
    picks = list(order[:n_each]) + list(order[-n_each:]) + list(order[len(order) // 2: len(order) // 2 + n_each])
    return sorted({int(b) for b in picks})


def test_cfg1_every_output():
    batch = inputs.make_batch(inputs.CONFIGS["cfg1"], "cuda", poison=True)
    out = gpu_attention(batch)
    mx, mean = assert_parity(out, oracle_attention(batch).out, what="cfg1")
    print(f"cfg1 max abs {mx:.3e} mean abs {mean:.3e}")


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4"])
def test_large_config_sampled_sequences(name):
    cfg = inputs.CONFIGS[name]
    batch = inputs.make_batch(cfg, "cuda", poison=True)
    out = gpu_attention(batch)
    assert torch.isfinite(out.float()).all()
    seqs = sample_sequences(batch.context_lens)
    ref = oracle_attention(batch, seqs=seqs)
    mx, mean = assert_parity(out, ref.out, rows=seqs, what=name)
    print(f"{name} sampled {len(seqs)} sequences: max abs {mx:.3e} mean abs {mean:.3e}")
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
        ref1 = oracle_attention(batch, context_lens=lens1, seqs=seqs[:4])
        assert_parity(out1, ref1.out, rows=seqs[:4], what="cfg4 after append")
