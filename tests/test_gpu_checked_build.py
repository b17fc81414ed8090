"""The checked build (the library compiled with -DOOCO_CHECKS) on well-formed inputs.

Its kernels range-check every index they derive from device data and every shared-memory destination
of an asynchronous copy, and report violations in the status word instead of trapping.  No memory
checker can be run on these machines, so this is what stands guard over stray indices: the small
parity configurations, the 8-bit and several-query-token cases and the seeded random shapes run
through it here and must leave the status word at zero (and still match the oracle).  Nothing here
feeds the device an input meant to trip a check; the predicates themselves are unit-tested on the
host (tests/test_abi_host.py).
"""
import pytest

from paper_2511_21862_b200 import binding, build

import test_gpu_fp8
import test_gpu_fuzz
import test_gpu_multi_query
import test_gpu_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _checked_library():
    build.build()
    previous = binding.use_library(build.build(checked=True))
    assert binding.checked_build()
    yield
    binding.use_library(previous)
    assert not binding.checked_build()


@pytest.mark.parametrize("cfg", test_gpu_parity.SMALL, ids=lambda c: c.name)
def test_small_parity_configs(cfg):
    test_gpu_parity.test_attention_matches_oracle(cfg)


@pytest.mark.parametrize("cfg", test_gpu_fp8.CASES, ids=lambda c: c.name)
def test_fp8_cases(cfg):
    test_gpu_fp8.test_attention_fp8_matches_oracle(cfg)


@pytest.mark.parametrize("seed", range(64))
def test_fuzz_seeds(seed):
    test_gpu_fuzz.test_random_case(seed)


@pytest.mark.parametrize("seed", range(32))
def test_chunk_fuzz_seeds(seed):
    test_gpu_fuzz.test_random_chunk_case(seed)


@pytest.mark.parametrize("cfg,Sq", test_gpu_multi_query.CASES + test_gpu_multi_query.CHUNK_CASES,
                         ids=lambda v: getattr(v, "name", str(v)))
def test_multi_query_and_prefill_chunk_cases(cfg, Sq):
    test_gpu_multi_query.run_case(cfg, Sq, seed=cfg.seed)


def test_fused_steps():
    test_gpu_multi_query.test_fused_step_mq()
    test_gpu_multi_query.test_fused_step_prefill_chunk(40, 1)
    test_gpu_multi_query.test_fused_step_mq_over_8bit_cache()


def test_fused_step_and_block_permutation():
    test_gpu_parity.test_block_permutation_and_rerun_are_bit_identical()
    test_gpu_parity.test_shared_prefix_blocks_are_legal()
