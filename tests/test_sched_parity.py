"""Host-side scheduler of the library (C ABI) vs the plain Python oracle: latencies to rounding,
decisions exactly (a decision may differ only where the two latencies straddle the bound by rounding)."""
import numpy as np
import pytest

from oracle import sched_oracle as so
from paper_2511_21862_b200 import build, sched
from test_oracle_sched_pins import GOLDEN

REL = 1e-12


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


MODELS = {
    "qwen2.5-7b": (28, 3584, 28, 4, 128, 18944, 152064, 2, 1, 1),
    "qwen2.5-72b-tp4": (80, 8192, 64, 8, 128, 29568, 152064, 2, 4, 1),
    "llama3-8b": (32, 4096, 32, 8, 128, 14336, 128256, 2, 1, 1),
    "mha-ungated-fp8": (12, 768, 12, 12, 64, 3072, 50304, 1, 2, 0),
}
HWS = {
    "a100-like": (250e12, 200e12, 60e12, 1.4e12, 1.3e12, 8e-3, 4e-3, 100e9),
    "b200-like": (1.4e15, 1.0e15, 300e12, 6.0e12, 6.5e12, 3e-3, 1.5e-3, 700e9),
}
PAIRS = [(m, h) for m in MODELS for h in HWS]


def both(mname, hname):
    return (so.Model(*MODELS[mname]), so.Hw(*HWS[hname])), (sched.Model(*MODELS[mname]), sched.Hw(*HWS[hname]))


@pytest.mark.parametrize("row", GOLDEN, ids=["A", "B", "C"])
def test_library_matches_hand_computation(row):
    m, h, lens, want = row
    r = sched.predict_decode_latency(sched.Model(*m.__dict__.values()), sched.Hw(*h.__dict__.values()), len(lens), sum(lens))
    got = [r["gemm"], r["attention"], r["comm"], r["total"], r["gemm_compute_bound"], r["attention_compute_bound"]]
    assert got == pytest.approx(want, rel=1e-14)


@pytest.mark.parametrize("mname,hname", PAIRS)
def test_latency_predictor(mname, hname):
    (om, oh), (lm, lh) = both(mname, hname)
    rng = np.random.default_rng(hash((mname, hname)) % 2**32)
    for n in [0, 1, 2, 7, 64, 300, 1000]:
        lens = rng.integers(1, 40000, n).tolist()
        want = so.predict_decode_latency(om, oh, lens)
        got = sched.predict_decode_latency(lm, lh, n, sum(lens))
        for k in ("total", "gemm", "attention", "comm", "overhead"):
            assert got[k] == pytest.approx(want[k], rel=REL, abs=0), (k, n)
        assert got["gemm_compute_bound"] == want["gemm_compute_bound"]
        assert got["attention_compute_bound"] == want["attention_compute_bound"]
    assert sched.compute_saturated_batch(lm, lh) == so.compute_saturated_batch(om, oh)


def decisions_agree(sel_lib, sel_or, relation_holds):
    """Equal, or the disagreement is a rounding tie on the bound (then both answers are valid)."""
    if list(sel_lib) == list(sel_or):
        return True
    return relation_holds()


@pytest.mark.parametrize("mname,hname", PAIRS)
def test_mix_decoding_selection(mname, hname):
    (om, oh), (lm, lh) = both(mname, hname)
    rng = np.random.default_rng(1 + hash((mname, hname)) % 2**32)
    for trial in range(12):
        on = rng.integers(100, 4000, rng.integers(0, 40)).tolist()
        off = rng.integers(300, 33000, rng.integers(0, 60)).tolist()
        if trial % 4 == 0 and off:
            off[0] = off[-1]                                  # equal lengths: order by index
        base = so.L(om, oh, on)
        S = base * rng.uniform(0.9 if trial == 5 else 1.01, 3.0)
        K = int(rng.integers(0, 8))
        draws = rng.integers(-1, max(1, len(off)) + 1, K + 2).tolist()   # repeats and out-of-range ids included
        want_sel, want_lat, want_over = so.mix_decoding_select(om, oh, on, off, S, draws, K)
        sel, lat, over = sched.mix_decoding_select(lm, lh, on, off, S, draws, K)
        assert sel.tolist() == want_sel, (trial, S)
        assert lat == pytest.approx(want_lat, rel=REL) and over == want_over


@pytest.mark.parametrize("mname,hname", PAIRS)
def test_migration_preference(mname, hname):
    import dataclasses
    (om, oh), (lm, lh) = both(mname, hname)
    om, lm = dataclasses.replace(om, num_layers=3), dataclasses.replace(lm, num_layers=3)   # keeps the oracle's scans short
    rng = np.random.default_rng(2 + hash((mname, hname)) % 2**32)
    sat = so.compute_saturated_batch(om, oh)
    for trial in range(8):
        n = int(rng.integers(1, min(2 * sat, sat + 40) if trial % 2 else max(2, sat // 2)))
        lens = rng.integers(50, 3000, n).tolist()
        base = so.L(om, oh, lens)
        S = base * rng.uniform(0.95 if trial == 3 else 1.005, 1.6)
        cap = int(sum(lens) * rng.uniform(1.0, 1.5)) + int(rng.integers(0, 3000))
        lo, hi = int(rng.integers(1, 200)), int(rng.integers(200, 500))
        inc = int(trial != 7)
        want = so.migration_length_preference(om, oh, lens, inc, S, sat, cap, lo, hi)
        got = sched.migration_length_preference(lm, lh, n, sum(lens), inc, S, sat, cap, lo, hi)
        assert got == want, (trial, n, sat)


def test_closest_evictions_fit_and_argument_errors():
    rng = np.random.default_rng(3)
    for trial in range(30):
        lens = rng.integers(1, 50, rng.integers(0, 25)).tolist()        # many ties
        pref, cnt = int(rng.integers(0, 60)), int(rng.integers(0, 30))
        assert sched.select_closest_to_preference(lens, pref, cnt) == so.select_closest_to_preference(lens, pref, cnt)
        need, cb = int(rng.integers(0, 400)), int(trial % 2)
        ev, freed = sched.select_evictions(lens, need, cb)
        wev, wfreed = so.select_evictions(lens, need, cb)
        assert ev.tolist() == wev and freed == wfreed
    xs = rng.uniform(1e8, 2e10, 9)
    ys = 9e-6 + xs / 6.9e12 * (1 + 0.01 * rng.standard_normal(9))
    M, O = sched.fit_bandwidth(xs, ys)
    wM, wO = so.fit_bandwidth(xs.tolist(), ys.tolist())
    assert M == pytest.approx(wM, rel=1e-10) and O == pytest.approx(wO, rel=1e-8)
    lm, lh = sched.Model(*MODELS["llama3-8b"]), sched.Hw(*HWS["a100-like"])
    with pytest.raises(Exception):
        sched.predict_decode_latency(sched.Model(2, 8, 3, 2, 4, 8, 8), lh, 1, 1)       # Hq % Hkv != 0
    with pytest.raises(Exception):
        sched.predict_decode_latency(lm, sched.Hw(0, 1, 1, 1, 1, 0, 0, 1), 1, 1)       # F_g = 0
    with pytest.raises(Exception):
        sched.fit_bandwidth([1.0, 1.0], [2.0, 3.0])                                     # one distinct x


@pytest.mark.parametrize("mname,hname", PAIRS)
def test_prefill_latency_predictor(mname, hname):
    (om, oh), (lm, lh) = both(mname, hname)
    rng = np.random.default_rng(4 + hash((mname, hname)) % 2**32)
    for n in [0, 1, 3, 17]:
        lens = rng.integers(1, 6000, n).tolist() + ([0, -3] if n == 3 else [])
        want = so.predict_prefill_latency(om, oh, lens)
        got = sched.predict_prefill_latency(lm, lh, lens)
        for k in ("total", "gemm", "attention", "comm", "overhead"):
            assert got[k] == pytest.approx(want[k], rel=REL, abs=0), (k, n)
