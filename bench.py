#!/usr/bin/env python
"""Benchmark of the paged decode path (KV append + paged GQA decode attention) on B200.

A "step" is one pass of the whole hot path for one transformer layer over one synthetic decode
batch: ooco_decode_step, i.e. the append of the new token's K/V fused into the plan launch, the
split-KV attention kernel and the LSE merge kernel (three launches).  Successive steps use different pool replicas (as successive layers of a
model do), so the KV working set of the timed region is far larger than L2.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl ours|reference]

Prints ONE JSON line.  The default workload is the largest long-context configuration (cfg4: 512 sequences of
1 K to 16 K tokens over a fragmented pool, with the append); at N = 1 the other full-size workloads are timed
in the same run and reported under `per_config`.  With N > 1 (under torchrun) every rank runs an independent replica of the
workload (its own seed); there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2511_21862_b200 import inputs

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
METRIC = "paged decode-attn achieved HBM TB/s"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    """Dense bf16 TFLOP/s (burst figure: the kernel is timed alone)."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return FALLBACK_BF16_TFLOPS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the benchmark runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.period, self.index = period_s, index
        self.samples = []          # (t, sm_mhz, reasons_bitmask, power_w)
        self._stop_evt = threading.Event()
        self.max_mhz = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    rs = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    rs = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                try:
                    pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                except Exception:
                    pw = None
                self.samples.append((time.perf_counter(), mhz, rs, pw))
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)

    def summary(self, t0, t1):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        win = [s for s in self.samples if t0 <= s[0] <= t1] or self.samples
        mhz = sorted(s[1] for s in win)
        bits = 0
        for s in win:
            bits |= s[2]
        names = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
                 0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
                 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
        reasons = [n for b, n in names.items() if bits & b]
        pw = [s[3] for s in win if s[3] is not None]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(win), "power_w_max": max(pw) if pw else None}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate(world, step_ms_local, units_local):
    """(max over ranks of the step time, sum over ranks of the units) -- gloo/nccl all-reduce."""
    if world == 1:
        return step_ms_local, units_local
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([step_ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def replica_count(pool_bytes: int, free_bytes: int) -> int:
    """Pool replicas so that the rotating KV working set is >= 4 GiB (>> the 126 MB L2)."""
    want = max(2, -(-(4 << 30) // max(1, pool_bytes)))
    fit = max(1, int(free_bytes * 0.6) // max(1, pool_bytes))
    return max(1, min(want, fit, 16))


def sample_bytes_of(cfg, tokens: int, nseq: int) -> int:
    """Model bytes (operator table, d = 2) of `nseq` whole sequences holding `tokens` cached tokens."""
    return tokens * 2 * 2 * cfg.num_kv_heads * cfg.head_dim + 2 * 2 * nseq * cfg.num_q_heads * cfg.head_dim


def run_reference(args, rank, world):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload per step.

    Only the sampled sequences' blocks are synthesised on the host (lengths and block-table rows are the
    full workload's own draws), so the largest workloads need no 20 GB host pool."""
    if rank != 0:
        return
    import numpy as np
    import oracle
    cfg = inputs.CONFIGS[args.workload]
    lens_all = inputs.draw_layout(cfg).lens.numpy()
    # sample: whole sequences, shortest first, up to ~budget tokens * heads per step
    budget = args.ref_token_heads
    order = np.argsort(lens_all, kind="stable")
    chosen, acc = [], 0
    for b in order:
        cost = int(lens_all[b]) * cfg.num_q_heads
        if chosen and acc + cost > budget:
            break
        chosen.append(int(b)); acc += cost
    batch = inputs.make_sample_batch(cfg, chosen, "cpu")
    lens = batch.context_lens.numpy()
    tok = int(lens.sum())
    sample_bytes = sample_bytes_of(cfg, tok, len(chosen))
    q, k, v = inputs.as_u16(batch.q), inputs.as_u16(batch.k_cache), inputs.as_u16(batch.v_cache)
    table = batch.block_table.numpy()

    def step():
        oracle.decode_attention(q, k, v, table, lens, cfg.scale, num_kv_heads=cfg.num_kv_heads,
                                block_size=cfg.block_size, strides=batch.strides)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    ms = dt / args.steps * 1e3
    val = sample_bytes / (ms * 1e-3) / 1e12
    sample = (f"{len(chosen)} shortest of the {len(lens_all)} sequences of {cfg.name} ({tok} tokens, all "
              f"{cfg.num_q_heads} q heads) per step")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "description": cfg.description, "sample": sample},
        "cpu_baseline": {"value": val, "unit": "TB/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "TB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
        "decode_tokens_per_s": len(chosen) / (ms * 1e-3),
    }
    print(json.dumps(line))


def cpu_baseline(cfg, batch, budget_s=12.0, max_sample_bytes=4 << 30):
    """Oracle timed on the host cores on a bounded sample of the same workload (rank 0, N = 1): whole
    sequences, longest first, at most `max_sample_bytes` of K + V, repeated for about `budget_s`.  The
    sample's blocks are compacted on the device and copied to the host; the oracle call is the stock one."""
    import numpy as np
    import oracle
    lens = batch.context_lens.cpu().numpy()
    table = batch.block_table.cpu()
    bs = cfg.block_size
    per_token = 2 * 2 * cfg.num_kv_heads * cfg.head_dim
    order = np.argsort(lens, kind="stable")[::-1]
    chosen, acc = [], 0
    for b in order:
        need = int(lens[b]) * per_token
        if chosen and acc + need > max_sample_bytes:
            continue
        chosen.append(int(b)); acc += need
    chosen.sort()
    ids, rows = [], []
    for b in chosen:
        n = (int(lens[b]) + bs - 1) // bs
        row = torch.zeros(table.shape[1], dtype=torch.int32)
        row[:n] = torch.arange(len(ids), len(ids) + n, dtype=torch.int32)
        ids.extend(table[b, :n].tolist())
        rows.append(row)
    idx = torch.tensor(ids if ids else [0], dtype=torch.long, device=batch.k_cache.device)
    k = inputs.as_u16(batch.k_cache.index_select(0, idx))
    v = inputs.as_u16(batch.v_cache.index_select(0, idx))
    q = inputs.as_u16(batch.q[chosen].contiguous())
    tab, ln = torch.stack(rows).numpy(), lens[chosen].astype(np.int32)

    def run():
        t0 = time.perf_counter()
        oracle.decode_attention(q, k, v, tab, ln, cfg.scale, num_kv_heads=cfg.num_kv_heads, block_size=bs,
                                strides=batch.strides)
        return time.perf_counter() - t0
    dt = run()
    reps = int(max(1, min(256, round(budget_s / max(dt, 1e-4)) - 1)))
    if reps > 1 or dt < 1.0:
        t0 = time.perf_counter()
        for _ in range(reps):
            run()
        dt = (time.perf_counter() - t0) / reps
    tok = int(ln.sum())
    return {"value": sample_bytes_of(cfg, tok, len(chosen)) / dt / 1e12, "unit": "TB/s", "cores": oracle.num_threads(),
            "kind": "oracle",
            "sample": f"{len(chosen)} of {len(lens)} sequences of {cfg.name} ({tok} of {int(lens.sum())} tokens, "
                      f"all q heads), {dt:.2f} s per pass x {reps}",
            "decode_tokens_per_s": len(chosen) / dt}


def kernel_source_digest() -> str:
    """Digest of the sources the attention kernel is compiled from (ncu counters taken on another
    version of them are not reported)."""
    import hashlib
    h = hashlib.sha256()
    for f in ("decode_kernels.cuh", "ptx.cuh"):
        with open(os.path.join(ROOT, "paper_2511_21862_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload: str, algorithmic_bytes: int):
    """(DRAM bytes read + written per launch of the attention kernel, how it was obtained) from the ncu
    figures recorded in profiles/decode_main_kernel_dram_traffic.txt, or (None, why).

    A workload with a capture of its own reports it; the others are scaled from the capture the file
    marks `scale_from`, by algorithmic bytes (traffic grows in proportion to the tokens read).  Lines:
    `source <digest>`, `capture <name> <dram bytes> <algorithmic bytes>`, `scale_from <name>`."""
    path = os.path.join(ROOT, "profiles", "decode_main_kernel_dram_traffic.txt")
    try:
        rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None, "no capture recorded"
    digest = next((r[1] for r in rows if r[0] == "source"), None)
    if digest != kernel_source_digest():
        return None, "kernel sources changed since the capture"
    caps = {r[1]: (int(r[2]), int(r[3])) for r in rows if r[0] == "capture"}
    if workload in caps:
        return caps[workload][0], f"ncu capture of {workload}"
    base = next((r[1] for r in rows if r[0] == "scale_from"), None)
    if base in caps:
        return int(round(caps[base][0] / caps[base][1] * algorithmic_bytes)), f"scaled from the ncu capture of {base}"
    return None, "no capture recorded"


def measure_workload(args, cfg, dev, rank, world, *, e2e=True, baseline=False):
    """Times one workload: K steps device-resident (value), the same K steps with events between the
    kernels (kernel_ms), and the host-buffer step (e2e).  Returns a dict of local (this rank's) figures."""
    from paper_2511_21862_b200 import binding
    if world > 1:
        import torch.distributed as dist
    batch = inputs.make_batch(cfg, dev, poison=False)
    fp8 = args.kv == "fp8"
    K_SCALE, V_SCALE = 1.0 / 32, 1.0 / 32                                 # N(0, sigma) values sit well inside +-448
    if fp8:
        batch = inputs.to_e4m3_pool(batch, K_SCALE, V_SCALE, poison=False)
    sh = binding.shape_of(batch)
    B = sh.batch
    lens_host = batch.context_lens.cpu().contiguous()
    lens1_host = (lens_host + 1).contiguous()                             # the step attends T_b + 1 tokens
    cost = binding.decode_bytes_model(sh, lens1_host)
    if fp8:                                                               # K / V stored with d = 1, q / out with d = 2
        cost = dict(cost, bytes_kv=binding.decode_bytes_model(sh, lens1_host, 1)["bytes_kv"])
        cost["bytes_paper"] = cost["bytes_q"] + cost["bytes_out"] + cost["bytes_kv"]
    kv_b = 1 if fp8 else 2
    append_bytes = 2 * B * cfg.num_kv_heads * cfg.head_dim * (2 + kv_b)   # K and V rows: bf16 read, cache written
    step_bytes = cost["bytes_paper"] + append_bytes

    pool_bytes = 2 * batch.k_cache.numel() * batch.k_cache.element_size()
    free, _ = torch.cuda.mem_get_info(dev)
    R = args.replicas if args.replicas > 0 else replica_count(pool_bytes, free)
    pools = [(batch.k_cache, batch.v_cache)] + [(batch.k_cache.clone(), batch.v_cache.clone()) for _ in range(R - 1)]
    ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device=dev)
    out = torch.empty_like(batch.q)
    positions = batch.context_lens                                        # append at T_b ...
    lens1 = (batch.context_lens + 1).contiguous()                         # ... then attend T_b + 1 tokens
    stream = torch.cuda.current_stream()

    def step(i):
        k, v = pools[i % R]
        if fp8:
            binding.decode_step_fp8(sh, batch.q, batch.k_new, batch.v_new, k, v, batch.block_table, positions, lens1,
                                    cfg.scale, K_SCALE, V_SCALE, out, ws, stream)
        else:
            binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, k, v, batch.block_table, positions, lens1,
                                cfg.scale, out, ws, stream)

    sampler = ClockSampler(dev.index)
    sampler.start()
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin = time.perf_counter()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t_end = time.perf_counter()
    ms_local = e0.elapsed_time(e1) / args.steps
    launches_per_step = binding.last_launch_count()                       # kernels of one timed step
    assert binding.workspace_status(ws) == 0
    clocks = sampler.summary(t_begin, t_end)

    # ---- per-kernel durations: the same K steps again with CUDA events recorded between the kernels on
    # the launching stream (the events switch off the programmatic launch overlap, so this pass is kept
    # out of the region `value` is taken from)
    binding.profile_enable(args.steps)
    for i in range(args.steps):
        step(i)
    recs = binding.profile_read(args.steps)
    binding.profile_enable(0)
    res = {"cfg": cfg, "B": B, "cost": cost, "step_bytes": step_bytes, "ms": ms_local, "recs": recs, "clocks": clocks,
           "R": R, "pool_bytes": pool_bytes, "launches_per_step": launches_per_step, "e2e_ms": None}

    # ---- end to end through the host-buffer entry point (pinned inputs in, result out, every step)
    if e2e and not fp8:
        pin = lambda t: t.cpu().contiguous().pin_memory()
        hq, hk, hv, ht = pin(batch.q), pin(batch.k_new), pin(batch.v_new), pin(batch.block_table)
        hp, hl = pin(positions), pin(lens1)
        hout = torch.empty(batch.q.shape, dtype=torch.bfloat16).pin_memory()
        stg = torch.empty(binding.step_staging_bytes(sh), dtype=torch.uint8, device=dev)
        res["h2d"] = sum(t.numel() * t.element_size() for t in (hq, hk, hv, ht, hp, hl))
        res["d2h"] = hout.numel() * hout.element_size()
        e2e_steps = max(3, min(args.steps, 200))

        def e2e_step(i):
            k, v = pools[i % R]
            binding.decode_step_host(sh, hq, hk, hv, ht, hp, hl, k, v, cfg.scale, hout, stg, ws, stream)
        for i in range(3):
            e2e_step(i)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        enq = wait = 0
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            e2e_step(i)
            a, b = binding.last_host_step_ns()
            enq, wait = enq + a, wait + b
        torch.cuda.synchronize()
        res["e2e_ms"] = (time.perf_counter() - t0) / e2e_steps * 1e3
        res["e2e_steps"] = e2e_steps
        # host time inside the call: until everything was enqueued / waiting for the stream (microseconds)
        res["e2e_host_us"] = {"enqueue": enq / e2e_steps / 1e3, "wait": wait / e2e_steps / 1e3}
    sampler.stop()
    if baseline:
        res["cpu_baseline"] = cpu_baseline(cfg, batch, args.cpu_seconds)
    return res


def roofline_of(res, peak, peak_kind):
    cost = res["cost"]
    attn_ms = sorted(r[1] for r in res["recs"])
    attn_avg = sum(attn_ms) / len(attn_ms)
    kernel_bytes = cost["bytes_kv"] + cost["bytes_q"] + cost["bytes_out"]
    achieved = kernel_bytes / (attn_avg * 1e-3) / 1e9
    traffic, how = ncu_traffic(res["cfg"].name, kernel_bytes) if res["cfg"].name in inputs.CONFIGS else (None, "no capture recorded")
    kernel_ms = {"plan": sum(r[0] for r in res["recs"]) / len(res["recs"]), "attention": attn_avg,
                 "attention_median": attn_ms[len(attn_ms) // 2], "merge": sum(r[2] for r in res["recs"]) / len(res["recs"])}
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_kind": f"of {peak_kind}", "frac_of_nominal_8tbps": achieved / NOMINAL_HBM_GBS,
            "kernel": "decode_main_kernel", "algorithmic_bytes_per_launch": kernel_bytes,
            "traffic": traffic, "traffic_source": how}
    return kernel_ms, roof


def run_ours(args, rank, local_rank, world):
    from paper_2511_21862_b200 import binding, build
    build.build()
    binding.lib()
    for kv in args.knob:
        name, val = kv.split("=")
        binding.set_tuning(**{name: int(val)})
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    cfg = inputs.replace(inputs.CONFIGS[args.workload], seed=inputs.CONFIGS[args.workload].seed + 100 * rank)
    if args.batch_div > 1 or args.len_div > 1:                            # a smaller sibling (profiler captures)
        cfg = inputs.scaled_config(cfg, batch_div=args.batch_div, len_div=args.len_div)
        cfg = inputs.replace(cfg, description=cfg.description + f" [batch / {args.batch_div}, lengths / {args.len_div}]")
    if args.block_size:                                                   # the same sequences over a pool of other blocks
        cfg = inputs.replace(cfg, block_size=args.block_size, name=f"{cfg.name}-bs{args.block_size}",
                             description=cfg.description + f" [block size overridden: {args.block_size}]")
    fp8 = args.kv == "fp8"
    res = measure_workload(args, cfg, dev, rank, world, e2e=True,
                           baseline=world == 1 and not args.no_cpu_baseline and not fp8)
    if fp8:
        return finish_fp8(args, world, cfg, res["B"], res["cost"], res["step_bytes"], res["ms"], res["recs"],
                          res["clocks"], res["R"], res["pool_bytes"])
    B, cost, step_bytes, R, pool_bytes = res["B"], res["cost"], res["step_bytes"], res["R"], res["pool_bytes"]
    ms, total_bytes = aggregate(world, res["ms"], float(step_bytes))
    e2e_ms, _ = aggregate(world, res["e2e_ms"], 0.0)
    _, total_seqs = aggregate(world, 0.0, float(B))
    # the other full-size workloads, timed the same way in the same run (N = 1 only)
    per_config = {}
    peak, peak_kind = measured_peak()
    if world == 1 and not args.no_per_config and not args.block_size and args.batch_div == 1 and args.len_div == 1:
        torch.cuda.empty_cache()
        for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
            if name == args.workload:
                continue
            torch.cuda.empty_cache()
            sub = argparse.Namespace(**vars(args))
            sub.steps = args.steps if name in ("cfg2", "cfg4") else 5 * args.steps   # short steps: a longer timed region
            r = measure_workload(sub, inputs.CONFIGS[name], dev, rank, world, e2e=True, baseline=False)
            km, roof = roofline_of(r, peak, peak_kind)
            v = r["step_bytes"] / (r["ms"] * 1e-3) / 1e12
            per_config[name] = {
                "step_TBps": v, "ms_per_step": r["ms"], "steps": sub.steps, "pct_of_nominal_8tbps": 100.0 * v * 1e3 / NOMINAL_HBM_GBS,
                "pct_of_measured_copy": 100.0 * v * 1e3 / peak, "kernel_ms": km,
                "kernel_GBps": roof["achieved"], "kernel_frac_of_measured": roof["frac"],
                "kernel_frac_of_nominal_8tbps": roof["frac_of_nominal_8tbps"], "traffic": roof["traffic"],
                "traffic_source": roof["traffic_source"], "e2e_ms_per_step": r["e2e_ms"], "e2e_host_us_per_call": r["e2e_host_us"],
                "total_tokens": r["cost"]["total_tokens"], "batch": r["B"], "pool_replicas": r["R"], "clocks": r["clocks"]}
    if rank != 0:
        return
    value = total_bytes / (ms * 1e-3) / 1e12
    kernel_ms, roof = roofline_of(res, peak, peak_kind)
    line = {
        "metric": METRIC, "value": value, "unit": "TB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "description": cfg.description, "batch": B,
                   "total_tokens": cost["total_tokens"], "step": "ooco_decode_step: fused kv append + plan, split-KV attention, LSE merge; one layer",
                   "l2": f"inputs larger than L2: steps rotate over {R} pool replica(s) ({R * pool_bytes / 2**30:.2f} GiB), "
                         f"{cost['bytes_kv'] / 2**30:.2f} GiB of K + V read per step",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "pct_of_nominal_8tbps": 100.0 * value * 1e3 / (NOMINAL_HBM_GBS * world),
        "pct_of_measured_copy": 100.0 * value * 1e3 / (peak * world),
        "decode_tokens_per_s": total_seqs / (ms * 1e-3),
        "step_bytes": step_bytes,
        "kernel_ms": kernel_ms,
        "roofline": roof,
        "e2e": {"value": total_bytes / (e2e_ms * 1e-3) / 1e12, "unit": "TB/s", "h2d_bytes_per_step": res["h2d"],
                "d2h_bytes_per_step": res["d2h"], "ms_per_step": e2e_ms, "steps": res["e2e_steps"],
                "host_us_per_call": res["e2e_host_us"]},
        "gpu_launches": args.steps * res["launches_per_step"],
        "clocks": res["clocks"],
    }
    if per_config:
        line["per_config"] = per_config
    if "cpu_baseline" in res:
        line["cpu_baseline"] = res["cpu_baseline"]
    print(json.dumps(line))


def run_block_moves(args, rank, local_rank, world):
    """Secondary measurement: paged KV block movement (the data movement of a request migration).

    One step packs the blocks of `--move-seqs` sequences of the workload (longest first) into a
    contiguous buffer and unpacks them into free blocks of a second pool; gather and scatter are also
    timed alone.  Successive steps use other pool replicas / packed buffers (working set >> L2)."""
    from paper_2511_21862_b200 import binding, build
    build.build()
    binding.lib()
    for kv in args.knob:
        name, val = kv.split("=")
        binding.set_tuning(**{name: int(val)})
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    cfg = inputs.CONFIGS[args.workload]
    batch = inputs.make_batch(cfg, dev, poison=False)
    sh = binding.shape_of(batch)
    lens, table = batch.context_lens.cpu(), batch.block_table.cpu()
    order = torch.argsort(lens, descending=True)[: args.move_seqs].tolist()
    bs = cfg.block_size
    ids = torch.cat([table[b, : (int(lens[b]) + bs - 1) // bs] for b in order]).contiguous()
    n = ids.numel()
    block_bytes = 2 * cfg.num_kv_heads * bs * cfg.head_dim * 2             # K + V words of one block
    moved = n * block_bytes
    R = max(2, min(8, -(-(1 << 30) // moved)))
    gen = torch.Generator().manual_seed(cfg.seed + 9)
    dst_ids = [torch.randperm(batch.num_blocks, generator=gen)[:n].to(torch.int32).to(dev) for _ in range(R)]
    ids_d = ids.to(dev)
    words = n * cfg.num_kv_heads * bs * cfg.head_dim
    packs = [(torch.empty(words, dtype=torch.bfloat16, device=dev), torch.empty(words, dtype=torch.bfloat16, device=dev))
             for _ in range(R)]
    pool2 = (torch.empty_like(batch.k_cache), torch.empty_like(batch.v_cache))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def gather(i):
        binding.kv_gather_blocks(sh, batch.k_cache, batch.v_cache, ids_d, *packs[i % R], status, stream)

    def scatter(i):
        binding.kv_scatter_blocks(sh, *packs[i % R], dst_ids[i % R], *pool2, status, stream)

    def timed(fn, steps):
        for i in range(args.warmup):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    sampler = ClockSampler(local_rank)
    sampler.start()
    t0 = time.perf_counter()
    ms_g = timed(gather, args.steps)
    ms_s = timed(scatter, args.steps)
    ms_both = timed(lambda i: (gather(i), scatter(i)), args.steps)
    t1 = time.perf_counter()
    sampler.stop()
    assert int(status.item()) == 0
    peak, peak_kind = measured_peak()
    gbs = lambda ms: 2 * moved / (ms * 1e-3) / 1e9                          # bytes read + bytes written
    line = {
        "metric": "paged KV block movement GB/s (read + written)", "value": gbs(ms_both / 2), "unit": "GB/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_both, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: migrate the {len(order)} longest sequences", "blocks": n,
                   "bytes_moved": moved, "step": "ooco_kv_gather_blocks then ooco_kv_scatter_blocks",
                   "l2": f"inputs larger than L2: {R} packed buffers / destination lists rotated"},
        "kernel_ms": {"gather": ms_g, "scatter": ms_s, "gather_then_scatter": ms_both},
        "roofline": {"bound": "hbm", "achieved": gbs(ms_g), "peak": peak, "unit": "GB/s", "frac": gbs(ms_g) / peak,
                     "peak_kind": f"of {peak_kind}", "kernel": "block_copy_kernel (gather)",
                     "algorithmic_bytes_per_launch": 2 * moved, "traffic": None,
                     "scatter": {"achieved": gbs(ms_s), "frac": gbs(ms_s) / peak}},
        "gpu_launches": 2 * args.steps, "clocks": sampler.summary(t0, t1),
    }
    print(json.dumps(line))


def run_multi_query(args, local_rank):
    """Secondary measurement: several query tokens per sequence (multi-token decode).  One step appends
    q_len new tokens per sequence and attends with causal masking over the cache (ooco_decode_step_mq).  Bytes follow the operator table with S_q = q_len."""
    from paper_2511_21862_b200 import binding, build
    build.build()
    binding.lib()
    for kv in args.knob:
        name, val = kv.split("=")
        binding.set_tuning(**{name: int(val)})
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()
    Sq = args.q_len
    base = inputs.CONFIGS[args.workload]
    cfg = inputs.replace(base, groups=tuple(inputs.replace(g, lo=g.lo + Sq, hi=g.hi + Sq) if g.dist != "fixed" else g
                                            for g in base.groups))
    batch = inputs.make_batch(cfg, dev, poison=False)
    fp8 = args.kv == "fp8"
    KS = VS = 1.0 / 32
    if fp8:
        batch = inputs.to_e4m3_pool(batch, KS, VS, poison=False)
    sh = binding.shape_of(batch)
    B = sh.batch
    gen = torch.Generator(device=dev).manual_seed(cfg.seed + 7)
    q = (torch.randn((B, Sq, cfg.num_q_heads, cfg.head_dim), generator=gen, device=dev) * cfg.sigma).to(torch.bfloat16)
    k_new = (torch.randn((B, Sq, cfg.num_kv_heads, cfg.head_dim), generator=gen, device=dev) * cfg.sigma).to(torch.bfloat16)
    v_new = (torch.randn((B, Sq, cfg.num_kv_heads, cfg.head_dim), generator=gen, device=dev) * cfg.sigma).to(torch.bfloat16)
    positions = (batch.context_lens - Sq).contiguous()                   # the new tokens are the last q_len of each context
    lens_host = batch.context_lens.cpu().contiguous()
    cost = binding.attention_bytes_model(sh, Sq, lens_host)                     # table row with S_q = q_len
    if fp8:                                                                     # K / V stored with d = 1
        cost = dict(cost, bytes_kv=cost["bytes_kv"] // 2)
        cost["bytes_paper"] = cost["bytes_q"] + cost["bytes_out"] + cost["bytes_kv"]
    nbytes = cost["bytes_paper"]
    pool_bytes = 2 * batch.k_cache.numel() * batch.k_cache.element_size()
    free, _ = torch.cuda.mem_get_info(dev)
    R = replica_count(pool_bytes, free)
    pools = [(batch.k_cache, batch.v_cache)] + [(batch.k_cache.clone(), batch.v_cache.clone()) for _ in range(R - 1)]
    ws = torch.empty(binding.workspace_bytes_mq(sh, Sq), dtype=torch.uint8, device=dev)
    out = torch.empty_like(q)

    def step(i):
        k, v = pools[i % R]
        if fp8:
            binding.decode_step_mq_fp8(sh, q, k_new, v_new, k, v, batch.block_table, positions, batch.context_lens,
                                       cfg.scale, KS, VS, out, ws, stream)
        else:
            binding.decode_step_mq(sh, q, k_new, v_new, k, v, batch.block_table, positions, batch.context_lens,
                                   cfg.scale, out, ws, stream)
    sampler = ClockSampler(local_rank)
    sampler.start()
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    assert binding.workspace_status(ws) == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    binding.profile_enable(args.steps)
    for i in range(args.steps):
        step(i)
    recs = binding.profile_read(args.steps)
    binding.profile_enable(0)
    attn = sum(r[1] for r in recs) / len(recs)
    peak, peak_kind = measured_peak()
    achieved = nbytes / (attn * 1e-3) / 1e9
    columns = Sq * (cfg.num_q_heads // cfg.num_kv_heads)
    knobs = dict(k.split("=", 1) for k in args.knob)
    tc_knob, tt_knob = int(knobs.get("chunk_tcgen05", 1)), int(knobs.get("chunk_two_tiles", 2))
    tc_from = 17 if tc_knob == 1 else tc_knob                              # first column count on the tcgen05 kernels
    tcgen05 = columns > 16 and cfg.head_dim == 128 and (fp8 or (tc_knob != 0 and columns >= tc_from))
    two_tiles = tcgen05 and tt_knob != 0 and ((columns <= 128 and tt_knob == 2) if fp8 else (columns > 128 or tt_knob == 2))
    kernel = (("chunk_tc2_kernel" if two_tiles else "chunk_tc_kernel") if tcgen05 else "chunk_main_kernel") if columns > 16 else (
        "row16_main_kernel" if columns > 8 and not fp8 else "decode_main_kernel")   # (the 8-bit cache has no row16 kernel)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind}", "kernel": kernel, "algorithmic_bytes_per_launch": nbytes,
                "traffic": None}
    # Eq. "op_latency": the operator is bound by whichever of FLOPs / F and bytes / M is larger
    tf_peak, tf_kind = measured_tensor_peak()
    tflops = cost["flops"] / (attn * 1e-3) / 1e12
    if cost["flops"] / (tf_peak * 1e12) > nbytes / (peak * 1e9):
        roofline = {"bound": "tensor", "achieved": tflops, "peak": tf_peak, "unit": "TFLOP/s", "frac": tflops / tf_peak,
                    "peak_kind": f"of {tf_kind} (bf16 GEMM burst)", "kernel": kernel,
                    "algorithmic_flops_per_launch": cost["flops"], "traffic": None,
                    "note": "flops as the operator table prints them (no causal discount)"}
    print(json.dumps({
        "metric": METRIC + f" ({Sq} query tokens per sequence" + (", 8-bit E4M3 KV cache)" if fp8 else ")"), "value": nbytes / (ms * 1e-3) / 1e12, "unit": "TB/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16 (e4m3 codes widened)" if fp8 else "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}, {Sq} query tokens per sequence" + (", 8-bit cache" if fp8 else ""), "batch": B,
                   "total_tokens": cost["total_tokens"], "step": "ooco_decode_step_mq, one layer",
                   "l2": f"inputs larger than L2: steps rotate over {R} pool replicas"},
        "query_tokens_per_s": B * Sq / (ms * 1e-3),
        "kernel_ms": {"plan": sum(r[0] for r in recs) / len(recs), "attention": attn, "merge": sum(r[2] for r in recs) / len(recs)},
        "attention_tflops": tflops, "roofline": roofline,
        "gpu_launches": 3 * args.steps, "clocks": sampler.summary(t0, t1)}))


def run_serve_loop(args, local_rank):
    """Secondary measurement: the step-level scheduling of a latency-strict instance driving the kernels.

    An attention-only instance (one layer) decodes all its online requests every step and, beside them, the
    offline requests Algorithm "Mix Decoding Selection" admits under the TPOT bound S; after each step
    Algorithm "Offline Request Migration Decision" may pull offline requests of the preferred length from a
    pool of candidates (a latency-relaxed instance), online requests arrive and leave, and when the KV pool
    is full offline requests are evicted by the rule of section 3.4.1.  Every step is one
    ooco_decode_step_host call (block tables, lengths and new rows come from host memory); its wall time
    is what is compared with S.  The latency predictor uses M_a and the overhead fitted on a few
    host-step measurements taken first; the bound handed to the algorithms carries a 3 % margin and a running
    measured / predicted correction."""
    import numpy as np
    from paper_2511_21862_b200 import binding, build, sched
    build.build()
    binding.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()
    rng = np.random.default_rng(2024)
    Hq, Hkv, D, bs = 40, 8, 128, 16                                        # the cfg2 shape
    scale = 1.0 / math.sqrt(D)
    cap_tokens = args.pool_tokens
    NB = cap_tokens // bs
    MB = (32768 + 2048) // bs
    Bmax = 640
    g = torch.Generator(device=dev).manual_seed(9)
    k_cache = (torch.randn((NB, Hkv, bs, D), generator=g, device=dev)).to(torch.bfloat16)
    v_cache = (torch.randn((NB, Hkv, bs, D), generator=g, device=dev)).to(torch.bfloat16)
    pin = lambda t: t.pin_memory()
    hq = pin(torch.randn((Bmax, Hq, D)).to(torch.bfloat16))
    hk = pin(torch.randn((Bmax, Hkv, D)).to(torch.bfloat16))
    hv = pin(torch.randn((Bmax, Hkv, D)).to(torch.bfloat16))
    htab = pin(torch.zeros((Bmax, MB), dtype=torch.int32))
    hpos = pin(torch.zeros(Bmax, dtype=torch.int32))
    hlen = pin(torch.zeros(Bmax, dtype=torch.int32))
    hout = pin(torch.empty((Bmax, Hq, D), dtype=torch.bfloat16))
    free_blocks = list(rng.permutation(NB))

    class Req:
        __slots__ = ("len", "left", "blocks", "online")

        def __init__(self, length, left, online):
            self.len, self.left, self.online, self.blocks = int(length), int(left), online, []

    def reserve(r, tokens):                                                # blocks for `tokens` cached tokens
        need = -(-tokens // bs) - len(r.blocks)
        if need > len(free_blocks):
            return False
        for _ in range(max(0, need)):
            r.blocks.append(free_blocks.pop())
        return True

    def release(r):
        free_blocks.extend(r.blocks)
        r.blocks = []

    def run_step(batch):
        B = len(batch)
        tab = htab.numpy()
        for i, r in enumerate(batch):
            tab[i, :len(r.blocks)] = r.blocks
            hpos[i] = r.len
            hlen[i] = r.len + 1
        sh = binding.Shape(B, Hq, Hkv, D, bs, NB, MB, Hkv * bs * D, bs * D, D)
        ws = ws_all[: binding.workspace_bytes(sh)]
        stg = stg_all[: binding.step_staging_bytes(sh)]
        t0 = time.perf_counter()
        binding.decode_step_host(sh, hq[:B], hk[:B], hv[:B], htab[:B], hpos[:B], hlen[:B], k_cache, v_cache, scale,
                                 hout[:B], stg, ws, stream)
        return time.perf_counter() - t0

    sh_max = binding.Shape(Bmax, Hq, Hkv, D, bs, NB, MB, Hkv * bs * D, bs * D, D)
    ws_all = torch.empty(binding.workspace_bytes(sh_max), dtype=torch.uint8, device=dev)
    stg_all = torch.empty(binding.step_staging_bytes(sh_max), dtype=torch.uint8, device=dev)

    # ---- profiling data for the predictor: a few batches through the same host-step call
    xs, ys = [], []
    for nreq, lo, hi in ((32, 512, 4096), (96, 2048, 8192), (160, 4096, 16384), (64, 8192, 32768), (256, 4096, 12000),
                         (48, 512, 2048), (128, 1024, 6000)):
        reqs = [Req(rng.integers(lo, hi), 1, False) for _ in range(nreq)]
        while sum(r.len + bs for r in reqs) > 0.9 * cap_tokens:           # a small pool: fewer requests
            reqs.pop()
        assert all(reserve(r, r.len + 1) for r in reqs)
        nreq = len(reqs)
        for _ in range(3):
            run_step(reqs)
        t = min(run_step(reqs) for _ in range(10))
        sh = binding.Shape(nreq, Hq, Hkv, D, bs, NB, MB, Hkv * bs * D, bs * D, D)
        cost = binding.decode_bytes_model(sh, torch.tensor([r.len + 1 for r in reqs], dtype=torch.int32))
        xs.append(cost["bytes_paper"]); ys.append(t)
        for r in reqs:
            release(r)
    M_a, O = sched.fit_bandwidth(xs, ys)
    model = sched.Model(1, Hq * D, Hq, Hkv, D, D, D)
    big = 1e30
    hw = sched.Hw(big, big, big, big, M_a, 0.0, O, big)
    bs_sat = 256                                                           # an instance parameter (compute-saturated batch)

    # ---- the instance
    S = args.slo_ms * 1e-3
    margin = 0.97
    corr = 1.0                                                             # running measured / predicted ratio
    online = [Req(rng.integers(512, 4097), rng.integers(50, 300), True) for _ in range(32)]
    for r in online:
        assert reserve(r, r.len + 1)
    offline = []
    new_offline = lambda: Req(int(np.exp(rng.uniform(np.log(4096), np.log(32768)))), rng.integers(100, 1000), False)
    relaxed_pool = [new_offline() for _ in range(400)]
    stats = {"steps": 0, "within": 0, "batch": 0, "offline_tokens": 0, "evicted": 0, "migrated": 0, "worst_ms": 0.0,
             "sum_ms": 0.0, "online_tokens": 0, "pred_err": 0.0}
    t_begin = time.perf_counter()
    for step_i in range(args.steps):
        on_lens = [r.len + 1 for r in online]
        off_lens = [r.len + 1 for r in offline]
        K = 8
        probes = rng.permutation(len(offline))[:K].tolist() if offline else []
        sel, pred, over = sched.mix_decoding_select(model, hw, on_lens, off_lens, S * margin / corr, probes, len(probes))
        chosen = [r for r, m in zip(offline, sel) if m]
        batch = online + chosen
        # room for the token of this step; when the pool runs dry, offline requests are evicted by the rule
        # of section 3.4.1 (they go back to the latency-relaxed side and leave this step's batch)
        while True:
            short = sum(1 for r in batch if len(r.blocks) * bs < r.len + 1) - len(free_blocks)
            if short <= 0:
                break
            ev, freed = sched.select_evictions([x.len for x in offline], (short + 32) * bs, len(batch) >= bs_sat)
            assert ev.any(), "KV pool exhausted by online requests alone"
            for x, e in zip(list(offline), ev):
                if e:
                    release(x); offline.remove(x); relaxed_pool.append(x); stats["evicted"] += 1
                    if x in chosen:
                        chosen.remove(x)
            batch = online + chosen
        for r in batch:
            assert reserve(r, r.len + 1)
        sec = run_step(batch)
        stats["steps"] += 1
        stats["within"] += sec <= S
        stats["batch"] += len(batch)
        stats["sum_ms"] += sec * 1e3
        stats["worst_ms"] = max(stats["worst_ms"], sec * 1e3)
        stats["pred_err"] += abs(pred - sec) / sec
        corr = 0.9 * corr + 0.1 * min(1.5, max(0.67, sec / pred))         # feedback on the predictor's bias
        stats["offline_tokens"] += len(chosen)
        stats["online_tokens"] += len(online)
        for r in batch:
            r.len += 1
            r.left -= 1
        for r in [r for r in online if r.left <= 0]:                       # finished online requests leave, new ones arrive
            release(r); online.remove(r)
            n = Req(rng.integers(512, 4097), rng.integers(50, 300), True)
            need = -(-(n.len + 1) // bs)
            if need > len(free_blocks):                                    # section 3.4.1: evict offline requests to make room
                ev, freed = sched.select_evictions([x.len for x in offline], (need - len(free_blocks)) * bs,
                                                   len(batch) >= bs_sat)
                for x, e in zip(list(offline), ev):
                    if e:
                        release(x); offline.remove(x); relaxed_pool.append(x); stats["evicted"] += 1
            assert reserve(n, n.len + 1)
            online.append(n)
        for r in [r for r in offline if r.left <= 0]:
            release(r); offline.remove(r); relaxed_pool.append(new_offline())
        # migration decision (pull model): only when everything on the instance already decodes
        tokens = sum(r.len for r in batch)
        pref = sched.migration_length_preference(model, hw, len(batch), tokens, len(chosen) == len(offline), S * margin / corr,
                                                 bs_sat, cap_tokens - 64 * bs, 4096, 32768)
        if pref >= 0 and relaxed_pool:
            picks = sched.select_closest_to_preference([r.len for r in relaxed_pool], pref, 4)
            for idx in sorted(picks, reverse=True):
                r = relaxed_pool[idx]
                headroom = 2 * (len(batch) + 4)                            # blocks the residents will need soon
                if -(-(r.len + 1) // bs) + headroom <= len(free_blocks) and reserve(r, r.len + 1):
                    offline.append(relaxed_pool.pop(idx)); stats["migrated"] += 1
    wall = time.perf_counter() - t_begin
    n = stats["steps"]
    print(json.dumps({
        "metric": "latency-strict instance loop: share of decode steps within the TPOT bound", "value": stats["within"] / n,
        "unit": "fraction", "higher_is_better": True, "n_gpus": 1, "steps": n, "data": "synthetic", "dtype": "bf16",
        "config": {"workload": "32 online requests U[512,4096] + offline requests log-uniform [4096,32768] pulled by "
                               "the migration decision; cfg2 head shape; one layer", "slo_ms": args.slo_ms,
                   "margin": margin, "pool_tokens": cap_tokens, "bs_sat": bs_sat},
        "fitted": {"M_a_GBps": M_a / 1e9, "overhead_us": O * 1e6},
        "mean_step_ms": stats["sum_ms"] / n, "worst_step_ms": stats["worst_ms"], "mean_batch": stats["batch"] / n,
        "mean_abs_prediction_error": stats["pred_err"] / n,
        "offline_tokens_per_s_of_gpu_time": stats["offline_tokens"] / (stats["sum_ms"] * 1e-3),
        "online_tokens_per_s_of_gpu_time": stats["online_tokens"] / (stats["sum_ms"] * 1e-3),
        "slo_utilisation": stats["sum_ms"] / n / args.slo_ms, "migrated": stats["migrated"], "evicted": stats["evicted"],
        "offline_resident_at_end": len(offline), "host_loop_wall_s": wall}))


def run_model_fit(args, local_rank):
    """Secondary measurement: the attention term of the Roofline latency model against this kernel.

    Profiling set: decode steps on reduced copies of the workloads (fewer sequences, shorter contexts).
    ooco_fit_bandwidth turns (model bytes, measured seconds) into the achievable bandwidth M_a and a
    static overhead; the fitted line then predicts the four full-size workloads, whose measured step
    times give the prediction error (the paper reports about 5 % for its whole-model predictor)."""
    from paper_2511_21862_b200 import binding, build, sched
    build.build()
    binding.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()

    def measure(cfg, steps, context_lens=None):
        batch = inputs.make_batch(cfg, dev, poison=False, context_lens=context_lens)
        sh = binding.shape_of(batch)
        cost = binding.decode_bytes_model(sh, batch.context_lens.cpu().contiguous())
        pool_bytes = 2 * batch.k_cache.numel() * 2
        free, _ = torch.cuda.mem_get_info(dev)
        R = replica_count(pool_bytes, free)
        pools = [(batch.k_cache, batch.v_cache)] + [(batch.k_cache.clone(), batch.v_cache.clone()) for _ in range(R - 1)]
        ws = torch.empty(binding.workspace_bytes(sh), dtype=torch.uint8, device=dev)
        out = torch.empty_like(batch.q)
        lens1 = (batch.context_lens + 1).contiguous()

        def step(i):
            k, v = pools[i % R]
            binding.decode_step(sh, batch.q, batch.k_new, batch.v_new, k, v, batch.block_table, batch.context_lens,
                                lens1, cfg.scale, out, ws, stream)
        for i in range(max(3, args.warmup)):
            step(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            step(i)
        e1.record(stream)
        torch.cuda.synchronize()
        assert binding.workspace_status(ws) == 0
        return cost, e0.elapsed_time(e1) / steps * 1e-3

    train, test = [], []
    for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
        base = inputs.CONFIGS[name]
        for bdiv, ldiv in ((4, 4), (2, 2), (4, 1)):
            cfg = inputs.scaled_config(base, batch_div=bdiv, len_div=ldiv)
            cost, sec = measure(cfg, 200)
            train.append({"workload": cfg.name, "bytes": cost["bytes_paper"], "tokens": cost["total_tokens"], "seconds": sec})
    M_a, O = sched.fit_bandwidth([r["bytes"] for r in train], [r["seconds"] for r in train])
    errs = []
    for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
        cost, sec = measure(inputs.CONFIGS[name], 100 if name in ("cfg2", "cfg4") else 400)
        pred = O + cost["bytes_paper"] / M_a
        errs.append(abs(pred - sec) / sec)
        test.append({"workload": name, "bytes": cost["bytes_paper"], "tokens": cost["total_tokens"], "seconds": sec,
                     "predicted": pred, "abs_rel_err": errs[-1]})
    # ---- closing the loop: Algorithm "Mix Decoding Selection" driven by the fitted predictor.  An
    # attention-only instance (one layer, GEMM terms switched off by unbounded F_g / M_g) gets a TPOT
    # bound S; the selection picks offline requests next to all online ones; the selected batch is
    # then actually run and its measured step time compared with S and with the prediction.
    base = inputs.CONFIGS["cfg2"]
    model = sched.Model(1, base.num_q_heads * base.head_dim, base.num_q_heads, base.num_kv_heads, base.head_dim,
                        base.head_dim, base.head_dim)
    big = 1e30
    hw = sched.Hw(big, big, big, big, M_a, 0.0, O, big)
    gen = torch.Generator().manual_seed(123)
    online = torch.randint(512, 4097, (32,), generator=gen).tolist()
    u = torch.rand(600, generator=gen, dtype=torch.float64)
    offline = torch.exp(math.log(4096) + u * (math.log(32768) - math.log(4096))).round().to(torch.int64).tolist()
    slo = []
    for S in (0.4e-3, 0.8e-3, 1.6e-3):
        K = 16
        probes = torch.randperm(len(offline), generator=gen)[:K].tolist()
        margin = 0.97                                                    # the predictor is good to a few percent
        sel, pred, over = sched.mix_decoding_select(model, hw, online, offline, S * margin, probes, K)
        lens = online + [t for t, m in zip(offline, sel) if m]
        cfg = inputs.replace(base, name=f"slo-{S * 1e3:.1f}ms", seed=77)
        batch_lens = torch.tensor(lens, dtype=torch.int32)
        cost, sec = measure(cfg, 100, context_lens=batch_lens)
        slo.append({"slo_ms": S * 1e3, "online": len(online), "offline_selected": int(sel.sum()), "margin": margin, "batch": len(lens),
                    "tokens": cost["total_tokens"], "predicted_ms": pred * 1e3, "measured_ms": sec * 1e3,
                    "within_slo": bool(sec <= S), "headroom": 1.0 - sec / S})
    line = {"metric": "Roofline attention-latency model: mean abs relative error on the full workloads",
            "value": sum(errs) / len(errs), "unit": "fraction", "higher_is_better": False, "n_gpus": 1,
            "M_a_GBps": M_a / 1e9, "overhead_us": O * 1e6, "profiling_set": train, "validation": test,
            "mix_decoding_selection": slo,
            "data": "synthetic", "dtype": "bf16"}
    print(json.dumps(line))


def finish_fp8(args, world, cfg, B, cost, step_bytes, ms, recs, clocks, R, pool_bytes):
    """JSON line of the 8-bit-cache variant (single GPU; device-resident inputs only)."""
    peak, peak_kind = measured_peak()
    attn = sorted(r[1] for r in recs)
    attn_avg = sum(attn) / len(attn)
    achieved = cost["bytes_paper"] / (attn_avg * 1e-3) / 1e9
    line = {
        "metric": METRIC + " (8-bit E4M3 KV cache)", "value": step_bytes / (ms * 1e-3) / 1e12, "unit": "TB/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16 (e4m3 codes widened)", "data": "synthetic",
        "config": {"workload": cfg.name + " with an 8-bit KV cache", "description": cfg.description, "batch": B,
                   "total_tokens": cost["total_tokens"], "step": "ooco_decode_step_fp8, one layer",
                   "l2": f"inputs larger than L2: steps rotate over {R} pool replicas ({R * pool_bytes / 2**30:.2f} GiB)"},
        "decode_tokens_per_s": B / (ms * 1e-3), "step_bytes": step_bytes,
        "kernel_ms": {"plan": sum(r[0] for r in recs) / len(recs), "attention": attn_avg,
                      "merge": sum(r[2] for r in recs) / len(recs)},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "kernel": "decode_main_kernel (8-bit cache)",
                     "algorithmic_bytes_per_launch": cost["bytes_paper"], "traffic": None},
        "gpu_launches": args.steps * 3, "clocks": clocks,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(inputs.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="time only --workload, not the other full-size workloads")
    ap.add_argument("--block-size", type=int, default=0, choices=[0, 16, 32, 64, 128, 256],
                    help="decode_step: KV block size instead of the workload's own (a sensitivity measurement; 0: keep)")
    ap.add_argument("--batch-div", type=int, default=1, help="decode_step: divide the workload's sequence counts (a smaller sibling)")
    ap.add_argument("--len-div", type=int, default=1, help="decode_step: divide the workload's context lengths")
    ap.add_argument("--replicas", type=int, default=0, help="pool replicas the steps rotate over (0: enough for 4 GiB)")
    ap.add_argument("--knob", action="append", default=[], help="launch-shape override name=value (sweeps)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--ref-token-heads", type=int, default=4_000_000,
                    help="reference arm: (tokens x q heads) of oracle work per step")
    ap.add_argument("--op", default="decode_step", choices=["decode_step", "kv_migrate", "model_fit", "decode_mq", "serve_loop"],
                    help="decode_step: the decode hot path (default); kv_migrate: paged block gather + scatter; "
                         "model_fit: fit and validate the attention term of the latency model; "
                         "decode_mq: --q-len query tokens per sequence; serve_loop: scheduler-driven decode loop")
    ap.add_argument("--slo-ms", type=float, default=1.0, help="serve_loop: TPOT bound of the one-layer instance")
    ap.add_argument("--pool-tokens", type=int, default=3_000_000, help="serve_loop: KV pool capacity in tokens")
    ap.add_argument("--q-len", type=int, default=4, help="decode_mq: query tokens per sequence")
    ap.add_argument("--kv", default="bf16", choices=["bf16", "fp8"],
                    help="decode_step: KV cache element type (fp8 = E4M3 codes; a secondary measurement)")
    ap.add_argument("--move-seqs", type=int, default=64, help="kv_migrate: sequences whose blocks are moved")
    args = ap.parse_args()
    rank, local_rank, world = dist_env()
    if args.op == "serve_loop":
        if rank == 0:
            args.steps = args.steps if args.steps is not None else 600
            run_serve_loop(args, local_rank)
        return
    if args.op == "decode_mq":
        if rank == 0:
            args.steps = args.steps if args.steps is not None else 300
            args.warmup = max(3, args.warmup if args.warmup is not None else 10)
            run_multi_query(args, local_rank)
        return
    if args.op == "model_fit":
        if rank == 0:
            args.warmup = args.warmup if args.warmup is not None else 5
            run_model_fit(args, local_rank)
        return
    if args.op == "kv_migrate":
        if rank == 0:
            args.steps = args.steps if args.steps is not None else 200
            args.warmup = max(3, args.warmup if args.warmup is not None else 10)
            run_block_moves(args, rank, local_rank, world)
        return
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 5
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args, rank, world)
        return
    args.steps = args.steps if args.steps is not None else (2000 if args.workload in ("cfg0", "cfg1") else 200)
    args.warmup = max(3, args.warmup if args.warmup is not None else 20)
    run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
