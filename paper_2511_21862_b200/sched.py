"""ctypes binding of the host-side scheduler ABI (`include/ooco_sched.h`): argument marshalling only."""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np

from .binding import OocoError, lib

SCHED_EXPORTS = (
    "ooco_predict_decode_latency", "ooco_compute_saturated_batch", "ooco_mix_decoding_select",
    "ooco_migration_length_preference", "ooco_select_closest_to_preference", "ooco_select_evictions",
    "ooco_fit_bandwidth", "ooco_predict_prefill_latency",
)


class ooco_hw_params_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("F_g", "F_ap", "F_ad", "M_g", "M_a", "O_p", "O_d", "B_c")]


class ooco_model_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("num_layers", "hidden", "num_q_heads", "num_kv_heads", "head_dim",
                                              "intermediate", "vocab", "bytes_per_value", "tp", "gated_mlp")]


class ooco_latency_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("total", "gemm", "attention", "comm", "overhead")] + \
               [(n, ctypes.c_int32) for n in ("gemm_compute_bound", "attention_compute_bound")]


@dataclass(frozen=True)
class Hw:
    F_g: float
    F_ap: float
    F_ad: float
    M_g: float
    M_a: float
    O_p: float
    O_d: float
    B_c: float

    def c(self):
        return ooco_hw_params_t(self.F_g, self.F_ap, self.F_ad, self.M_g, self.M_a, self.O_p, self.O_d, self.B_c)


@dataclass(frozen=True)
class Model:
    num_layers: int
    hidden: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    intermediate: int
    vocab: int
    bytes_per_value: int = 2
    tp: int = 1
    gated_mlp: int = 1

    def c(self):
        return ooco_model_t(self.num_layers, self.hidden, self.num_q_heads, self.num_kv_heads, self.head_dim,
                            self.intermediate, self.vocab, self.bytes_per_value, self.tp, self.gated_mlp)


_ready = False


def _lib():
    global _ready
    L = lib()
    if not _ready:
        mp, hp = ctypes.POINTER(ooco_model_t), ctypes.POINTER(ooco_hw_params_t)
        vp, i32, i64, f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        L.ooco_predict_decode_latency.restype = ctypes.c_int
        L.ooco_predict_decode_latency.argtypes = [mp, hp, i64, i64, ctypes.POINTER(ooco_latency_t)]
        L.ooco_predict_prefill_latency.restype = ctypes.c_int
        L.ooco_predict_prefill_latency.argtypes = [mp, hp, vp, i32, ctypes.POINTER(ooco_latency_t)]
        L.ooco_compute_saturated_batch.restype = i64
        L.ooco_compute_saturated_batch.argtypes = [mp, hp]
        L.ooco_mix_decoding_select.restype = ctypes.c_int
        L.ooco_mix_decoding_select.argtypes = [mp, hp, vp, i32, vp, i32, f64, vp, i32, vp, ctypes.POINTER(i32),
                                               ctypes.POINTER(f64), ctypes.POINTER(i32)]
        L.ooco_migration_length_preference.restype = ctypes.c_int
        L.ooco_migration_length_preference.argtypes = [mp, hp, i64, i64, i32, f64, i64, i64, i32, i32,
                                                       ctypes.POINTER(i32)]
        L.ooco_select_closest_to_preference.restype = ctypes.c_int
        L.ooco_select_closest_to_preference.argtypes = [vp, i32, i32, i32, vp, ctypes.POINTER(i32)]
        L.ooco_select_evictions.restype = ctypes.c_int
        L.ooco_select_evictions.argtypes = [vp, i32, i64, i32, vp, ctypes.POINTER(i64)]
        L.ooco_fit_bandwidth.restype = ctypes.c_int
        L.ooco_fit_bandwidth.argtypes = [vp, vp, i32, ctypes.POINTER(f64), ctypes.POINTER(f64)]
        _ready = True
    return L


def _check(rc, where):
    if rc != 0:
        raise OocoError(rc, where)


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32).reshape(-1))


def _p(a):
    return a.ctypes.data if a.size else None


def predict_decode_latency(model: Model, hw: Hw, batch_size: int, total_tokens: int) -> dict:
    out = ooco_latency_t()
    _check(_lib().ooco_predict_decode_latency(ctypes.byref(model.c()), ctypes.byref(hw.c()), int(batch_size),
                                              int(total_tokens), ctypes.byref(out)), "ooco_predict_decode_latency")
    return {n: getattr(out, n) for n, _ in ooco_latency_t._fields_}


def predict_prefill_latency(model: Model, hw: Hw, prompt_lens) -> dict:
    lens = _i32(prompt_lens)
    out = ooco_latency_t()
    _check(_lib().ooco_predict_prefill_latency(ctypes.byref(model.c()), ctypes.byref(hw.c()), _p(lens), lens.size,
                                               ctypes.byref(out)), "ooco_predict_prefill_latency")
    return {n: getattr(out, n) for n, _ in ooco_latency_t._fields_}


def compute_saturated_batch(model: Model, hw: Hw) -> int:
    n = int(_lib().ooco_compute_saturated_batch(ctypes.byref(model.c()), ctypes.byref(hw.c())))
    if n <= 0:
        raise OocoError(-2, "ooco_compute_saturated_batch")
    return n


def mix_decoding_select(model: Model, hw: Hw, online_lens, offline_lens, slo_seconds, probe_order, K=None):
    """(selected uint8 [n_off], latency of the selected batch, online-alone-over-SLO flag)."""
    on, off, pr = _i32(online_lens), _i32(offline_lens), _i32(probe_order)
    K = pr.size if K is None else min(int(K), pr.size)
    sel = np.zeros(off.size, dtype=np.uint8)
    nsel, lat, over = ctypes.c_int32(0), ctypes.c_double(0), ctypes.c_int32(0)
    _check(_lib().ooco_mix_decoding_select(ctypes.byref(model.c()), ctypes.byref(hw.c()), _p(on), on.size, _p(off),
                                           off.size, float(slo_seconds), _p(pr), K, _p(sel), ctypes.byref(nsel),
                                           ctypes.byref(lat), ctypes.byref(over)), "ooco_mix_decoding_select")
    assert int(sel.sum()) == nsel.value
    return sel, lat.value, over.value


def migration_length_preference(model: Model, hw: Hw, batch_size, total_tokens, all_included, slo_seconds, bs_sat,
                                capacity_tokens, len_min, len_max) -> int:
    pref = ctypes.c_int32(0)
    _check(_lib().ooco_migration_length_preference(
        ctypes.byref(model.c()), ctypes.byref(hw.c()), int(batch_size), int(total_tokens), int(bool(all_included)),
        float(slo_seconds), int(bs_sat), int(capacity_tokens), int(len_min), int(len_max), ctypes.byref(pref)),
        "ooco_migration_length_preference")
    return pref.value


def select_closest_to_preference(offline_lens, pref, count):
    off = _i32(offline_lens)
    out = np.zeros(max(1, min(max(0, int(count)), off.size)), dtype=np.int32)
    n = ctypes.c_int32(0)
    _check(_lib().ooco_select_closest_to_preference(_p(off), off.size, int(pref), int(count), out.ctypes.data,
                                                    ctypes.byref(n)), "ooco_select_closest_to_preference")
    return out[: n.value].tolist()


def select_evictions(offline_lens, need_tokens, compute_bound):
    off = _i32(offline_lens)
    ev = np.zeros(off.size, dtype=np.uint8)
    freed = ctypes.c_int64(0)
    _check(_lib().ooco_select_evictions(_p(off), off.size, int(need_tokens), int(bool(compute_bound)), _p(ev),
                                        ctypes.byref(freed)), "ooco_select_evictions")
    return ev, freed.value


def fit_bandwidth(nbytes, seconds):
    x = np.ascontiguousarray(np.asarray(nbytes, dtype=np.float64))
    y = np.ascontiguousarray(np.asarray(seconds, dtype=np.float64))
    assert x.size == y.size
    M, O = ctypes.c_double(0), ctypes.c_double(0)
    _check(_lib().ooco_fit_bandwidth(x.ctypes.data, y.ctypes.data, x.size, ctypes.byref(M), ctypes.byref(O)),
           "ooco_fit_bandwidth")
    return M.value, O.value
