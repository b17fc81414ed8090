"""Plain Python oracle of the Roofline latency model and the scheduling algorithms (TEST
INFRASTRUCTURE ONLY: imported by tests and the benchmark's baseline legs, never by the product).

Everything is written the slow, literal way: the latency predictor walks every operator of every
layer and adds their times one by one (section 3.3: "summing the latency of all operators within
the iteration and adding this overhead term"); the selection algorithms re-evaluate the predictor
from scratch for every candidate set and use linear scans where the algorithms say "largest".
All arithmetic is Python float (fp64) on exact integer FLOP / byte counts.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class Hw:
    """Table "Parameters for latency modeling"."""
    F_g: float
    F_ap: float
    F_ad: float
    M_g: float
    M_a: float
    O_p: float
    O_d: float
    B_c: float


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


def gemm_cost(N, D_in, D_out, d):
    """Table "Operator Modeling", GEMM row: (FLOPs, bytes)."""
    return 2 * N * D_in * D_out, d * (N * D_in + D_in * D_out + N * D_out)


def attention_cost(D_h, S_q, S_kv, H_q, H_kv, d):
    """Table "Operator Modeling", attention row, with the K/V width read as D_h * H_kv / H_q
    (the printed H_q / H_kv would make grouped-query attention read more than multi-head
    attention, against section 2.3; both agree at H_q = H_kv)."""
    assert (S_kv * D_h * H_kv) % H_q == 0
    return 4 * D_h * S_q * S_kv, 2 * d * (S_q * D_h + S_kv * D_h * H_kv // H_q)


def op_latency(flops, nbytes, F, M):
    """Eq. "op_latency"."""
    return max(flops / F, nbytes / M)


def decode_operators(model: Model, lens):
    """Every operator of one decode iteration, in execution order, as (kind, flops, bytes).
    The attention operator of a layer is one fused operator over the batch: its counts are the
    table's, summed over the requests (S_q = 1, S_kv = the request's cached tokens)."""
    m, d, tp = model, model.bytes_per_value, model.tp
    N = len(lens)
    ops = []
    if N == 0:
        return ops
    hq, hkv = m.num_q_heads // tp, m.num_kv_heads // tp
    D_h = hq * m.head_dim
    for _ in range(m.num_layers):
        ops.append(("gemm",) + gemm_cost(N, m.hidden, (hq + 2 * hkv) * m.head_dim, d))
        fl = by = 0
        for T in lens:
            f, b = attention_cost(D_h, 1, T, hq, hkv, d)
            fl, by = fl + f, by + b
        ops.append(("attention", fl, by))
        ops.append(("gemm",) + gemm_cost(N, D_h, m.hidden, d))
        if tp > 1:
            ops.append(("comm", 0, N * m.hidden * d))
        ops.append(("gemm",) + gemm_cost(N, m.hidden, (2 if m.gated_mlp else 1) * m.intermediate // tp, d))
        ops.append(("gemm",) + gemm_cost(N, m.intermediate // tp, m.hidden, d))
        if tp > 1:
            ops.append(("comm", 0, N * m.hidden * d))
    ops.append(("gemm",) + gemm_cost(N, m.hidden, m.vocab // tp, d))
    return ops


def predict_decode_latency(model: Model, hw: Hw, lens) -> dict:
    """L(B): sum of the operator latencies of the iteration plus O_d (section 3.3.2)."""
    parts = {"gemm": 0.0, "attention": 0.0, "comm": 0.0}
    g_fl = g_by = a_fl = a_by = 0.0
    for kind, fl, by in decode_operators(model, [max(0, int(t)) for t in lens]):
        if kind == "gemm":
            parts["gemm"] += op_latency(fl, by, hw.F_g, hw.M_g)
            g_fl += fl / hw.F_g
            g_by += by / hw.M_g
        elif kind == "attention":
            parts["attention"] += op_latency(fl, by, hw.F_ad, hw.M_a)
            a_fl += fl / hw.F_ad
            a_by += by / hw.M_a
        else:
            parts["comm"] += by / hw.B_c
    total = parts["gemm"] + parts["attention"] + parts["comm"] + hw.O_d
    return dict(parts, overhead=hw.O_d, total=total, gemm_compute_bound=int(len(lens) > 0 and g_fl >= g_by),
                attention_compute_bound=int(len(lens) > 0 and a_fl >= a_by))


def L(model, hw, lens) -> float:
    return predict_decode_latency(model, hw, lens)["total"]


def prefill_operators(model: Model, prompt_lens):
    """Every operator of one prefill iteration over the given prompts, in execution order.  Linear
    layers see all prompt tokens (N = their sum); the attention operator of a layer is one fused
    operator over the requests with S_q = S_kv = the prompt length (the table has no causal discount);
    only the last token of each request goes through the LM head."""
    m, d, tp = model, model.bytes_per_value, model.tp
    lens = [int(t) for t in prompt_lens if int(t) > 0]
    ops = []
    if not lens:
        return ops
    N = sum(lens)
    hq, hkv = m.num_q_heads // tp, m.num_kv_heads // tp
    D_h = hq * m.head_dim
    for _ in range(m.num_layers):
        ops.append(("gemm",) + gemm_cost(N, m.hidden, (hq + 2 * hkv) * m.head_dim, d))
        fl = by = 0
        for S in lens:
            f, b = attention_cost(D_h, S, S, hq, hkv, d)
            fl, by = fl + f, by + b
        ops.append(("attention", fl, by))
        ops.append(("gemm",) + gemm_cost(N, D_h, m.hidden, d))
        if tp > 1:
            ops.append(("comm", 0, N * m.hidden * d))
        ops.append(("gemm",) + gemm_cost(N, m.hidden, (2 if m.gated_mlp else 1) * m.intermediate // tp, d))
        ops.append(("gemm",) + gemm_cost(N, m.intermediate // tp, m.hidden, d))
        if tp > 1:
            ops.append(("comm", 0, N * m.hidden * d))
    ops.append(("gemm",) + gemm_cost(len(lens), m.hidden, m.vocab // tp, d))
    return ops


def predict_prefill_latency(model: Model, hw: Hw, prompt_lens) -> dict:
    """Latency of a prefill iteration: operator latencies (attention against F_ap) plus O_p."""
    parts = {"gemm": 0.0, "attention": 0.0, "comm": 0.0}
    for kind, fl, by in prefill_operators(model, prompt_lens):
        if kind == "gemm":
            parts["gemm"] += op_latency(fl, by, hw.F_g, hw.M_g)
        elif kind == "attention":
            parts["attention"] += op_latency(fl, by, hw.F_ap, hw.M_a)
        else:
            parts["comm"] += by / hw.B_c
    return dict(parts, overhead=hw.O_p, total=parts["gemm"] + parts["attention"] + parts["comm"] + hw.O_p)


def compute_saturated_batch(model: Model, hw: Hw, limit=1 << 20) -> int:
    """Smallest N whose GEMMs are compute-bound as a whole (linear scan)."""
    for N in range(1, limit):
        if predict_decode_latency(model, hw, [1] * N)["gemm_compute_bound"]:
            return N
    return limit


def mix_decoding_select(model, hw, online_lens, offline_lens, S, probe_order, K):
    """Algorithm "Mix Decoding Selection"; the random draws are the caller's `probe_order`."""
    batch = list(online_lens)                                   # all online requests are included
    n_off = len(offline_lens)
    selected = [0] * n_off
    tested = [False] * n_off
    over = int(L(model, hw, batch) > S)
    for r in list(probe_order)[:max(0, K)]:
        if not (0 <= r < n_off) or tested[r]:
            continue
        tested[r] = True
        if L(model, hw, batch + [offline_lens[r]]) <= S:
            batch.append(offline_lens[r])
            selected[r] = 1
        # else: discarded
    rest = [r for r in range(n_off) if not tested[r]]
    if rest and L(model, hw, batch) < S:
        rest.sort(key=lambda r: (offline_lens[r], r))         # ascending request length
        best = 0
        for k in range(1, len(rest) + 1):                       # largest prefix, by definition
            if L(model, hw, batch + [offline_lens[r] for r in rest[:k]]) <= S:
                best = k
        for r in rest[:best]:
            selected[r] = 1
            batch.append(offline_lens[r])
    return selected, L(model, hw, batch), over


def migration_length_preference(model, hw, batch_lens, all_included, S, bs_sat, capacity_tokens, len_min, len_max):
    """Algorithm "Offline Request Migration Decision" up to the length preference; -1 = none."""
    batch = list(batch_lens)
    if not (L(model, hw, batch) < S and all_included):
        return -1
    tokens = sum(batch)
    if len(batch) >= bs_sat:
        fits = [l for l in range(len_min, len_max + 1)
                if L(model, hw, batch + [l]) <= S and (tokens + l) <= capacity_tokens]
        return max(fits) if fits else -1
    g = bs_sat - len(batch)
    if L(model, hw, batch + [len_min] * g) <= S:                # a group that reaches saturation fits
        return max(l for l in range(len_min, len_max + 1) if L(model, hw, batch + [l] * g) <= S)
    return len_min                                              # choose the shortest requests


def select_closest_to_preference(offline_lens, pref, count):
    order = sorted(range(len(offline_lens)), key=lambda r: (abs(offline_lens[r] - pref), offline_lens[r], r))
    return order[:max(0, count)]


def select_evictions(offline_lens, need_tokens, compute_bound):
    """Section 3.4.1: longest first on a compute-bound instance, shortest first otherwise."""
    n = len(offline_lens)
    order = sorted(range(n), key=(lambda r: (-offline_lens[r], r)) if compute_bound else (lambda r: (offline_lens[r], r)))
    evicted, freed = [0] * n, 0
    for r in order:
        if freed >= need_tokens:
            break
        evicted[r] = 1
        freed += offline_lens[r]
    return evicted, freed


def fit_bandwidth(nbytes, seconds):
    """Ordinary least squares of seconds = overhead + bytes / M."""
    n = len(nbytes)
    mx, my = sum(nbytes) / n, sum(seconds) / n
    sxx = sum((x - mx) ** 2 for x in nbytes)
    sxy = sum((x - mx) * (y - my) for x, y in zip(nbytes, seconds))
    slope = sxy / sxx
    return 1.0 / slope, my - slope * mx
