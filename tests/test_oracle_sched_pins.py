"""Pins of the scheduling oracle (latency model + selection algorithms): hand-computed values,
closed forms, an independent C routine for the attention bytes, and hand-solvable toy regimes."""
import math
import os

import numpy as np
import pytest

import oracle
from oracle import sched_oracle as so

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def read_golden():
    rows = []
    for line in open(os.path.join(ROOT, "tests", "golden", "latency_model.txt")):
        if line.startswith("#") or not line.strip():
            continue
        m, h, lens, want = (p.split() for p in line.split("|"))
        rows.append((so.Model(*map(int, m)), so.Hw(*map(float, h)), [int(x) for x in lens], [float(x) for x in want]))
    return rows


GOLDEN = read_golden()


@pytest.mark.parametrize("row", GOLDEN, ids=["A", "B", "C"])
def test_latency_matches_hand_computation(row):
    model, hw, lens, want = row
    r = so.predict_decode_latency(model, hw, lens)
    got = [r["gemm"], r["attention"], r["comm"], r["total"], r["gemm_compute_bound"], r["attention_compute_bound"]]
    assert got == pytest.approx(want, rel=1e-14)


def test_operator_table_rows():
    assert so.gemm_cost(3, 4, 5, 2) == (120, 94)
    assert so.attention_cost(8, 1, 10, 4, 2, 2) == (320, 192)
    # at Hq = Hkv the reading coincides with the printed 2d (Sq Dh + Skv Dh Hq/Hkv)
    for Dh, Sq, Skv, d in [(64, 1, 77, 2), (256, 3, 1000, 1)]:
        assert so.attention_cost(Dh, Sq, Skv, 8, 8, d)[1] == 2 * d * (Sq * Dh + Skv * Dh)
    assert so.op_latency(10, 100, 5, 10) == 10 and so.op_latency(100, 10, 5, 10) == 20


def test_attention_bytes_agree_with_the_c_byte_model():
    """The batch sums of the attention row equal what the (separately written) C byte model returns."""
    rng = np.random.default_rng(0)
    for Hq, Hkv, D in [(32, 8, 128), (40, 8, 128), (8, 8, 64), (64, 8, 128)]:
        lens = rng.integers(1, 5000, 17)
        fl = by = 0
        for T in lens:
            f, b = so.attention_cost(Hq * D, 1, int(T), Hq, Hkv, 2)
            fl, by = fl + f, by + b
        c = oracle.bytes_model(lens, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, block_size=16)
        assert (fl, by) == (c["flops"], c["bytes_paper"])


QWEN7B = so.Model(28, 3584, 28, 4, 128, 18944, 152064)
HW = so.Hw(F_g=250e12, F_ap=200e12, F_ad=60e12, M_g=1.4e12, M_a=1.3e12, O_p=8e-3, O_d=4e-3, B_c=100e9)


def test_memory_bound_closed_form_and_monotonicity():
    inf = float("inf")
    hw = so.Hw(inf, inf, inf, 2e12, 1e12, 0, 3e-3, 1)
    lens = [100, 2000, 31, 4096]
    ops = so.decode_operators(QWEN7B, lens)
    want = 3e-3 + sum(b for k, _, b in ops if k == "gemm") / 2e12 + sum(b for k, _, b in ops if k == "attention") / 1e12
    assert so.L(QWEN7B, hw, lens) == pytest.approx(want, rel=1e-12)
    assert so.L(QWEN7B, HW, []) == HW.O_d
    prev = so.L(QWEN7B, HW, [])
    batch = []
    for T in [5, 900, 17, 30000, 1, 256]:
        batch.append(T)
        cur = so.L(QWEN7B, HW, batch)
        assert cur > prev
        prev = cur
    assert so.L(QWEN7B, HW, [100, 200]) < so.L(QWEN7B, HW, [100, 201])


def test_gemm_ridge_batch_size():
    """For weight-dominated GEMMs the crossover sits near d * F_g / (2 * M_g) (roofline ridge), and
    below it the GEMM time does not change with the batch size (section 3.3.3)."""
    bs_sat = so.compute_saturated_batch(QWEN7B, HW)
    ridge = 2 * HW.F_g / (2 * HW.M_g)
    assert ridge <= bs_sat <= 1.15 * ridge
    g = lambda N: so.predict_decode_latency(QWEN7B, HW, [1] * N)["gemm"]
    assert g(64) / g(1) < 1.08                       # memory-bound: nearly constant
    assert g(4 * bs_sat) / g(2 * bs_sat) == pytest.approx(2.0, rel=0.02)   # compute-bound: proportional


def toy():
    """L(B) = total tokens (seconds) up to ~1e-20: only the attention FLOP term matters."""
    big = 1e30
    m = so.Model(2, 4, 2, 1, 2, 4, 4)
    return m, so.Hw(big, big, 4 * (2 * 2) * 2, big, big, 0, 0, big)


def test_mix_decoding_hand_example():
    m, hw = toy()
    assert so.L(m, hw, [3, 4]) == pytest.approx(7.0)
    S = 20 + 1e-9
    sel, lat, over = so.mix_decoding_select(m, hw, [10], [5, 3, 8, 2], S, [2], 1)
    assert sel == [0, 0, 1, 1] and lat == pytest.approx(20.0) and over == 0   # probe adds 8, then prefix {2}
    sel, _, _ = so.mix_decoding_select(m, hw, [10], [5, 3, 8, 2], S, [], 0)
    assert sel == [1, 1, 0, 1]                                                 # 2 + 3 + 5 fit, 8 does not
    sel, _, _ = so.mix_decoding_select(m, hw, [10], [5, 3, 8, 2], S, [2, 0, 1, 3], 4)
    assert sel == [0, 0, 1, 1]                                                 # 8 in, 5 out, 3 out, 2 in
    sel, _, _ = so.mix_decoding_select(m, hw, [10], [5, 3, 8, 2], S, [2, 2, 7, -1, 0], 2)
    assert sel == [0, 0, 1, 1]                                                 # K counts draws, repeats pass
    sel, lat, over = so.mix_decoding_select(m, hw, [15, 10], [1, 2], S, [0], 1)
    assert sel == [0, 0] and over == 1 and lat == pytest.approx(25.0)          # online alone exceeds S


def test_mix_decoding_result_is_feasible_and_prefix_maximal():
    rng = np.random.default_rng(5)
    for trial in range(20):
        on = rng.integers(200, 3000, rng.integers(1, 30)).tolist()
        off = rng.integers(500, 30000, rng.integers(1, 40)).tolist()
        S = so.L(QWEN7B, HW, on) * rng.uniform(1.02, 2.5)
        K = int(rng.integers(0, 6))
        probes = rng.permutation(len(off))[:K].tolist()
        sel, lat, over = so.mix_decoding_select(QWEN7B, HW, on, off, S, probes, K)
        chosen = on + [off[r] for r in range(len(off)) if sel[r]]
        assert over == 0 and lat == so.L(QWEN7B, HW, chosen) and lat <= S
        untested_left = sorted((off[r], r) for r in range(len(off)) if not sel[r] and r not in probes)
        if untested_left:                                   # the shortest one left out would break S
            assert so.L(QWEN7B, HW, chosen + [untested_left[0][0]]) > S
            assert all(off[r] <= untested_left[0][0] for r in range(len(off)) if sel[r] and r not in probes)


def test_migration_preference_hand_examples():
    m, hw = toy()
    pref = lambda batch, inc, S, sat, cap, lo, hi: so.migration_length_preference(m, hw, batch, inc, S, sat, cap, lo, hi)
    e = 1e-9
    assert pref([10, 10], 1, 50 + e, 2, 10**9, 1, 100) == 30       # saturated: longest under the SLO
    assert pref([10, 10], 1, 50 + e, 2, 45, 1, 100) == 25          # ... and under the memory capacity
    assert pref([10, 10], 1, 50 + e, 2, 10**9, 1, 28) == 28
    assert pref([10, 10], 1, 50 + e, 2, 20, 1, 100) == -1          # nothing fits in memory
    assert pref([10], 1, 50 + e, 3, 10**9, 1, 100) == 20           # group of 2 reaches saturation: 10 + 2 l <= 50
    assert pref([10], 1, 11 + e, 3, 10**9, 1, 100) == 1            # saturation out of reach: shortest
    assert pref([10, 10], 1, 20, 2, 10**9, 1, 100) == -1           # L(B) is not below S
    assert pref([10, 10], 0, 50, 2, 10**9, 1, 100) == -1           # requests were left out of B


def test_closest_evictions_and_fit():
    assert so.select_closest_to_preference([100, 900, 450, 520, 480], 500, 3) == [4, 3, 2]      # 480 and 520 tie: shorter first
    assert so.select_closest_to_preference([10, 30], 20, 5) == [0, 1]
    ev, freed = so.select_evictions([100, 900, 450, 520], 1000, compute_bound=1)
    assert ev == [0, 1, 0, 1] and freed == 1420                    # longest first: 900 + 520
    ev, freed = so.select_evictions([100, 900, 450, 520], 1000, compute_bound=0)
    assert ev == [1, 0, 1, 1] and freed == 1070                    # shortest first: 100 + 450 + 520
    assert so.select_evictions([5, 6], 100, 0) == ([1, 1], 11)
    assert so.select_evictions([5, 6], 0, 1) == ([0, 0], 0)
    xs = [1e8, 5e8, 2e9, 7e9]
    M, O = so.fit_bandwidth(xs, [12e-6 + x / 6.5e12 for x in xs])
    assert M == pytest.approx(6.5e12, rel=1e-9) and O == pytest.approx(12e-6, rel=1e-9)
    rng = np.random.default_rng(1)
    ys = [10e-6 + x / 7e12 * (1 + 0.02 * rng.standard_normal()) for x in xs]
    slope, icpt = np.polyfit(xs, ys, 1)
    M, O = so.fit_bandwidth(xs, ys)
    assert M == pytest.approx(1 / slope, rel=1e-9) and O == pytest.approx(icpt, rel=1e-6)


def test_prefill_latency_hand_example_and_compute_saturation():
    """Hand-worked: layers 1, hidden 4, Hq 2, Hkv 1, head_dim 2, intermediate 6 (gated), vocab 8, d 2; prompts 3
    and 5 (N = 8).  QKV 8x4->8: 512 FLOP, 2(32+32+64) = 256 B; attention D_h = 4: 4*4*(9+25) = 544 FLOP,
    2*2*(3*4 + 3*2) + 2*2*(5*4 + 5*2) = 72 + 120 = 192 B; O 4->4: 256 FLOP, 2(32+16+32) = 160 B; up 4->12: 768 FLOP,
    2(32+48+96) = 352 B; down 6->4: 384 FLOP, 2(48+24+32) = 208 B; head (2 last tokens) 4->8: 128 FLOP, 2(8+32+16) = 112 B.
    F_g 64, M_g 32, F_ap 16, M_a 16, O_p 0.25: gemm max(8,8)+max(4,5)+max(12,11)+max(6,6.5)+max(2,3.5) = 35;
    attention max(34, 12) = 34."""
    m = so.Model(1, 4, 2, 1, 2, 6, 8)
    hw = so.Hw(F_g=64, F_ap=16, F_ad=1, M_g=32, M_a=16, O_p=0.25, O_d=9, B_c=1)
    r = so.predict_prefill_latency(m, hw, [3, 5])
    assert (r["gemm"], r["attention"], r["comm"], r["total"]) == pytest.approx((35.0, 34.0, 0.0, 69.25), rel=1e-14)
    assert so.predict_prefill_latency(m, hw, [])["total"] == 0.25
    # section 3.3.3: beyond a few hundred tokens prefill is compute-bound (GEMM time proportional to tokens)
    g = lambda S: so.predict_prefill_latency(QWEN7B, HW, [S])["gemm"]
    assert g(4096) / g(2048) == pytest.approx(2.0, rel=0.02)
    assert g(16) / g(8) < 1.1
