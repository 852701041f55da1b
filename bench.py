"""Benchmark of the rank-r decode attention step (append one token, attend over the whole rank-r cache).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one pass of the decode hot path over one batch: project + append the new K/V row of every
sequence, project q, split-KV attention over all cached rank-r rows, cross-split combine and lift.
Rank 0 prints ONE JSON line.  With N > 1 (torchrun) every rank runs its own batch (the path shards by
sequence with no exchange), timings are the max over ranks.  `--impl reference` times the fp64 CPU
oracle on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2408_05646_b200 import synth

METRIC = "rank-r decode attention KV GB/s (B=16, n=32k, 7B layer; us/step alongside)"
UNIT = "GB/s"
FILL_CHUNK = 1024          # tokens per append call while filling the cache
# DRAM bytes moved per algorithmic byte by decode_splitkv_kernel, from an ncu capture of the B = 2 case of the
# headline workload (dram__bytes_read.sum + dram__bytes_write.sum = 679.5 MB for 671.1 MB of K'/V' rows; traffic
# grows in proportion to the number of units).  None whenever that kernel has changed since the capture.
DECODE_TRAFFIC_RATIO = 679.532 / 671.109


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), ("measured (MEASURED_PEAKS.json hbm_gbs): the rate of a device copy counting read + write "
                                     "bytes, not a read ceiling; a read-only stream can exceed it, so frac may read above 1. "
                                     "The number to hold against the >= 70 % of 8 TB/s target is frac_of_nominal_8TBs")
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def algorithmic_bytes(wl, ranks_k, ranks_v, n):
    """K' and V' rows that one decode step must read: B * n * sum_h (r_k + r_v) * element size."""
    es = 2 if wl.dtype == "bf16" else 4
    return wl.batch * n * (sum(ranks_k) + sum(ranks_v)) * es


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# the CPU oracle leg (also the --impl reference arm)
# ----------------------------------------------------------------------------------------------

QUANT_LEGS = ((4, 32), (3, 32))                   # (bits, group) of the quantised-cache entries of the workload table
VARIANT = {"alibi": False, "rope": False}   # --alibi / --rope: position schemes on both sides (decode workloads)
ROPE_BASE = 10000.0


def variant_slopes(wl):
    return synth.alibi_slopes(wl.n_heads) if VARIANT["alibi"] else None


def host_description() -> dict:
    """CPU model and core counts of the machine the oracle is timed on."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for ln in f:
                if ln.lower().startswith("model name"):
                    model = ln.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    try:
        usable = len(os.sched_getaffinity(0))
    except AttributeError:
        usable = os.cpu_count() or 1
    return {"cpu_model": model, "logical_cpus": os.cpu_count(), "usable_cpus": usable}


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_setup(wl, ranks_k, ranks_v, U_k, U_v, units, history=None):
    """Oracle state for the sampled (sequence, head) units: projects their whole history once.
    `history` maps (b, h) -> (k_rows, v_rows) [n, d_head] float64; if None it is drawn on the CPU (sequence 0 only)."""
    from oracle import eigen_attention as orc
    units = list(units)
    lay = orc.LayerOracle(wl.batch, wl.n_heads, wl.d_head, U_k, U_v, tracked=units, alibi_slopes=variant_slopes(wl),
                          rope={"base": ROPE_BASE, "interleaved": False} if VARIANT["rope"] else None)
    if history is None:
        W_k = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_K")
        W_v = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_V")
        dt = synth.torch_dtype(wl.dtype)
        for ci, c in enumerate(range(0, wl.context, FILL_CHUNK)):
            t = min(FILL_CHUNK, wl.context - c)
            k = synth.lowrank_rows(W_k, 1, t, wl.sigma, wl.index, "K", chunk=ci, dtype=dt).double().numpy()
            v = synth.lowrank_rows(W_v, 1, t, wl.sigma, wl.index, "V", chunk=ci, dtype=dt).double().numpy()
            for (b, h) in units:
                assert b == 0
                lay.append_unit_rows((0, h), k[0, :, h, :], v[0, :, h, :])
    else:
        for u in units:
            lay.append_unit_rows(u, history[u][0], history[u][1])
    lay.set_len(wl.context)
    return lay


def oracle_timed_steps(lay, wl, q, k_new, v_new, steps, warmup):
    """Times `steps` oracle decode steps (append the new row, attend) on the tracked units.
    Returns (seconds per step, outputs of the last step)."""
    n0 = wl.context
    times, out = [], None
    for i in range(warmup + steps):
        for u in lay.units:                                   # rewind to the fixed context length
            lay.Kp[u] = lay.Kp[u][:n0]
            lay.Vp[u] = lay.Vp[u][:n0]
        lay.set_len(n0)
        t0 = time.perf_counter()
        lay.append_kv(k_new, v_new)
        out = lay.decode(q)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    return sum(times) / len(times), out


def run_reference(args, wl):
    """The fp64 oracle as it stands on the host cores; each step covers a bounded sample of units."""
    ranks = synth.draw_ranks(wl.n_heads, wl.ranks, wl.index)
    U_k = synth.make_bases(wl.d_head, ranks, wl.index, "U_K")
    U_v = synth.make_bases(wl.d_head, ranks, wl.index, "U_V")
    sample_heads = list(range(wl.n_heads))                  # all heads of sequence 0
    lay = oracle_sample_setup(wl, ranks, ranks, U_k, U_v, [(0, h) for h in sample_heads])
    dt = synth.torch_dtype(wl.dtype)
    W_k = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_K")
    W_v = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_V")
    k_new = synth.lowrank_rows(W_k, wl.batch, 1, wl.sigma, wl.index, "K", chunk=10**6, dtype=dt).double().numpy()
    v_new = synth.lowrank_rows(W_v, wl.batch, 1, wl.sigma, wl.index, "V", chunk=10**6, dtype=dt).double().numpy()
    q = synth.gaussian_query(wl.batch, wl.n_heads, wl.d_head, wl.q_scale, wl.index, dtype=dt).double().numpy()
    steps = min(args.steps, 40)          # ~0.3 s of host work per step: keep the whole run to a minute
    sec, _ = oracle_timed_steps(lay, wl, q, k_new, v_new, steps, min(args.warmup, 5))
    es = 2 if wl.dtype == "bf16" else 4
    sample_bytes = (wl.context + 1) * sum(2 * ranks[h] for h in sample_heads) * es
    gbs = sample_bytes / sec / 1e9
    cores = blas_threads()
    sample = (f"{len(sample_heads)} of {wl.batch * wl.n_heads} (sequence, head) units per step "
              f"(all heads of sequence 0), full context {wl.context}+1; GB/s counts the same "
              f"{es}-byte rank-r elements as the GPU metric")
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 5), "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "n_heads": wl.n_heads, "d_head": wl.d_head,
                   "rank": list(wl.ranks), "context": wl.context, "sampled_units": len(sample_heads)},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# multi-rank plumbing (one process per GPU; the path shards by sequence, so ranks never exchange data)
# ----------------------------------------------------------------------------------------------

def rank_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(x: float, world: int, device) -> float:
    """The slowest rank's time: the only collective of the benchmark (timing, not data)."""
    if world == 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_rank: int, world: int, ms_per_step: float) -> float:
    """Weak scaling: every rank streams its own batch shard's cache; the job's rate is the sum."""
    return world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def rank_chunk_base(rank: int) -> int:
    """Offset of a rank's random sub-streams, so that batch shards hold different sequences."""
    return rank * 100000


# ----------------------------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------------------------

def shuffled_page_table(batch, n_max, page_rows, seed):
    """Every sequence gets n_max / page_rows pages drawn without replacement from the whole pool."""
    per = n_max // page_rows
    perm = np.random.default_rng(seed).permutation(batch * per)
    return [[int(x) for x in perm[b * per:(b + 1) * per]] for b in range(batch)]


def build_layer(wl, device, binding, keep_units=(), rank=0, page_rows=0):
    """Creates the layer and fills `context` rows through eigen_attn_append_kv.  Returns the layer, the
    bases, and for the (sequence, head) units in keep_units the raw K/V history as float64 arrays."""
    ranks = synth.draw_ranks(wl.n_heads, wl.ranks, wl.index)
    U_k = synth.make_bases(wl.d_head, ranks, wl.index, "U_K")
    U_v = synth.make_bases(wl.d_head, ranks, wl.index, "U_V")
    dt = synth.torch_dtype(wl.dtype)
    n_max = wl.context + 1
    if page_rows:
        n_max = (n_max + page_rows - 1) // page_rows * page_rows
    lay = binding.EigenAttnLayer(wl.batch, wl.n_heads, wl.d_head, n_max, dt, U_k, U_v, device=device)
    if page_rows:                                       # pages shuffled across the pool before the first row is written
        lay.set_page_table(shuffled_page_table(wl.batch, n_max, page_rows, synth.stream_seed(wl.index, "subset", 99)), page_rows)
    if VARIANT["alibi"]:
        lay.set_alibi(variant_slopes(wl))
    if VARIANT["rope"]:
        lay.set_rope(ROPE_BASE)
    W_k = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_K", device=device)
    W_v = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_V", device=device)
    hist = {u: ([], []) for u in keep_units}
    for ci, c in enumerate(range(0, wl.context, FILL_CHUNK)):
        t = min(FILL_CHUNK, wl.context - c)
        cid = ci + rank_chunk_base(rank)
        k = synth.lowrank_rows(W_k, wl.batch, t, wl.sigma, wl.index, "K", chunk=cid, dtype=dt, device=device)
        v = synth.lowrank_rows(W_v, wl.batch, t, wl.sigma, wl.index, "V", chunk=cid, dtype=dt, device=device)
        lay.append_kv(k, v)
        for (b, h) in keep_units:
            hist[(b, h)][0].append(k[b, :, h, :].double().cpu().numpy())
            hist[(b, h)][1].append(v[b, :, h, :].double().cpu().numpy())
    hist = {u: (np.concatenate(a), np.concatenate(b)) for u, (a, b) in hist.items()}
    k_new = synth.lowrank_rows(W_k, wl.batch, 1, wl.sigma, wl.index, "K", chunk=10**6, dtype=dt, device=device)
    v_new = synth.lowrank_rows(W_v, wl.batch, 1, wl.sigma, wl.index, "V", chunk=10**6, dtype=dt, device=device)
    q = synth.gaussian_query(wl.batch, wl.n_heads, wl.d_head, wl.q_scale, wl.index, dtype=dt, device=device)
    torch.cuda.synchronize(device)
    return lay, ranks, U_k, U_v, hist, q, k_new, v_new


def run_ours(args, wl):
    import torch.distributed as dist
    rank, world, local = rank_env()
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    from paper_2408_05646_b200 import build
    if rank == 0:
        build.build_library()
    if world > 1:
        dist.barrier()
    from paper_2408_05646_b200 import binding

    do_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline
    # the oracle's sample: 64 seeded (sequence, head) units with both corners, every rank and every sequence
    ranks0 = synth.draw_ranks(wl.n_heads, wl.ranks, wl.index)
    keep_units = synth.sample_units(wl.batch, wl.n_heads, ranks0, 64, wl.index)[:64] if do_cpu else []
    lay, ranks, U_k, U_v, hist, q, k_new, v_new = build_layer(wl, device, binding, keep_units, rank=rank)
    n0 = wl.context
    assert lay.len == n0
    stream = torch.cuda.current_stream(device)
    out = torch.empty_like(q)

    def step():
        lay.set_len(n0)
        lay.decode_step(q, k_new, v_new, out=out)

    def sync_all():
        torch.cuda.synchronize(device)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(device)

    # ---- device-resident timing, with per-step events around the split-KV kernel
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for e0, e1 in ev:           # create the underlying CUDA events
        e0.record(stream)
        e1.record(stream)
    for _ in range(args.warmup):
        step()
    sync_all()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = lay.launch_count()
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    t_start.record(stream)
    for i in range(args.steps):
        lay.set_decode_events(ev[i][0], ev[i][1])
        step()
    t_stop.record(stream)
    sync_all()
    lay.set_decode_events(None, None)
    launches = lay.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    lay.poll_status()
    ms_total = t_start.elapsed_time(t_stop)
    kern_ms = [a.elapsed_time(b) for a, b in ev]
    ms_total = max_over_ranks(ms_total, world, device)
    ms_step = ms_total / args.steps
    bytes_step = algorithmic_bytes(wl, ranks, ranks, n0 + 1)
    value = whole_job_gbs(bytes_step, world, ms_step)
    kern_avg_ms = sum(kern_ms) / len(kern_ms)
    peak, peak_src = measured_peaks()
    achieved = bytes_step / (kern_avg_ms * 1e-3) / 1e9

    # ---- end to end: host tensors in, host tensor out, through the C ABI
    # one pinned buffer holding q, k, v back to back: the library then sends them as a single copy
    hqkv = torch.stack([q.cpu(), k_new.cpu(), v_new.cpu()]).pin_memory()
    hq, hk, hv = hqkv[0], hqkv[1], hqkv[2]
    hout = torch.empty_like(hq).pin_memory()
    for _ in range(args.warmup):
        lay.set_len(n0)
        lay.decode_step_host(hq, hk, hv, hout)
    sync_all()
    t0 = time.perf_counter()
    e_start, e_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_start.record(stream)
    for _ in range(args.steps):
        lay.set_len(n0)
        lay.decode_step_host(hq, hk, hv, hout)
    e_stop.record(stream)
    sync_all()
    e2e_ms = e_start.elapsed_time(e_stop)
    e2e_ms = max_over_ranks(e2e_ms, world, device)
    e2e_ms_step = e2e_ms / args.steps
    e2e_value = whole_job_gbs(bytes_step, world, e2e_ms_step)
    io_bytes = hq.numel() * hq.element_size()
    same = bool(torch.equal(hout, out.cpu()))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- the oracle on the host cores: a bounded sample, also a full-size parity check
    cpu = None
    parity = None
    if do_cpu:
        ref = oracle_sample_setup(wl, ranks, ranks, U_k, U_v, keep_units, history=hist)
        del hist
        qn, kn, vn = q.double().cpu().numpy(), k_new.double().cpu().numpy(), v_new.double().cpu().numpy()
        sec, res = oracle_timed_steps(ref, wl, qn, kn, vn, steps=8, warmup=1)
        cores = blas_threads()
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            sec1, _ = oracle_timed_steps(ref, wl, qn, kn, vn, steps=2, warmup=1)
        es = 2 if wl.dtype == "bf16" else 4
        sample_bytes = (n0 + 1) * sum(2 * ranks[h] for _, h in keep_units) * es
        scale = wl.batch * wl.n_heads / len(keep_units)
        cpu = {"value": sample_bytes / sec / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
               "us_per_step_sample": sec * 1e6,
               "us_per_step_scaled_to_all_units": sec * 1e6 * scale,
               "one_thread": {"value": sample_bytes / sec1 / 1e9, "unit": UNIT, "cores": 1,
                              "us_per_step_sample": sec1 * 1e6, "us_per_step_scaled_to_all_units": sec1 * 1e6 * scale},
               "host": host_description(),
               "sample": f"{len(keep_units)} of {wl.batch * wl.n_heads} (sequence, head) units (seeded subset: both corners, "
                         f"every sequence), full context; a step = append the new row + attend; 8 timed steps with all "
                         f"BLAS threads, 2 with one thread; history projected beforehand"}
        g = out.double().cpu().numpy()
        errs = [np.abs(g[b, 0, h] - res[(b, h)]) for (b, h) in keep_units]
        parity = {"units": len(keep_units), "max_abs": float(max(e.max() for e in errs)),
                  "mean_abs": float(np.mean([e.mean() for e in errs])),
                  "tolerance": "max_abs <= 2e-2, mean_abs <= 2e-3 (bf16 storage)"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "us_per_step": ms_step * 1e3,
        "tokens_per_s": world * wl.batch / (ms_step * 1e-3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 storage, f32 accumulate" if wl.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "batch_per_gpu": wl.batch, "n_heads": wl.n_heads, "d_head": wl.d_head,
                   "rank": sorted(set(ranks)), "context": n0, "new_tokens": 1, "alibi": VARIANT["alibi"], "rope": VARIANT["rope"],
                   "cache_gb_per_gpu": bytes_step / 1e9, "parallelism": f"{world} independent batch shard(s)",
                   "l2": "inputs larger than L2: every step streams the whole rank-r cache"},
        "frac_of_nominal_8TBs": value / world / 8000.0,
        "roofline": {"bound": "hbm", "kernel": "decode_rope_kernel" if VARIANT["rope"] else "decode_splitkv_kernel", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                     "kernel_us": kern_avg_ms * 1e3, "algorithmic_bytes": bytes_step,
                     "traffic": (bytes_step * DECODE_TRAFFIC_RATIO
                                 if DECODE_TRAFFIC_RATIO and wl.name == "llama2_7b_b16_n32k" else None),
                     "traffic_source": "ncu dram bytes of the B=2 case scaled by units (profiles/)"},
        "e2e": {"value": e2e_value, "unit": UNIT, "us_per_step": e2e_ms_step * 1e3,
                "h2d_bytes_per_step": 3 * io_bytes, "d2h_bytes_per_step": io_bytes,
                "matches_device_path": same},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if not args.no_workloads and world == 1 and wl.name == "llama2_7b_b16_n32k" and not (VARIANT["alibi"] or VARIANT["rope"]):
        line["workloads"] = workload_table(device, binding, lay, wl, ranks, q, k_new, v_new)
        del lay
        torch.cuda.empty_cache()
        line["workloads"].update(workload_table_own_layers(device, binding))
        lay = None
    if not args.no_prefill and world == 1:
        del lay
        torch.cuda.empty_cache()
        line["prefill"] = prefill_measure(synth.WORKLOADS["prefill_b4_t4096"], device, steps=10, warmup=3)
        r = prefill_measure(synth.WORKLOADS["prefill_b4_t4096"], device, steps=10, warmup=3, rope=True)
        line["prefill_rope"] = {k: r[k] for k in ("workload", "ms_per_call", "attention_kernel_ms", "attention_tflops", "frac")}
        line["prefill_rope"]["what"] = ("the same prompt through a layer with rotary embedding: token rows projected, keys lifted "
                                        "and rotated, queries rotated, causal attention over d_head-wide rows; ms_per_call is all of it")
    if cpu is not None:
        line["cpu_baseline"] = cpu
        line["parity_full_size"] = parity
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def timed_kernel(lay, device, call, steps, warmup):
    """Runs `call()` warmup + steps times with the library's event pair around its attention kernel.
    Returns (median kernel us, mean us per call on the stream)."""
    stream = torch.cuda.current_stream(device)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        a.record(stream); b.record(stream)
    for _ in range(warmup):
        call()
    torch.cuda.synchronize(device)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for i in range(steps):
        lay.set_decode_events(ev[i][0], ev[i][1])
        call()
    t1.record(stream)
    torch.cuda.synchronize(device)
    lay.set_decode_events(None, None)
    lay.poll_status()
    ks = sorted(a.elapsed_time(b) for a, b in ev)
    return ks[len(ks) // 2] * 1e3, t0.elapsed_time(t1) / steps * 1e3


def table_entry(kernel, kernel_us, step_us, nbytes, peak, **extra):
    d = {"kernel": kernel, "kernel_us": round(kernel_us, 2), "step_us": round(step_us, 2), "algorithmic_bytes": int(nbytes),
         "GB/s": round(nbytes / kernel_us / 1e3, 1), "frac": round(nbytes / kernel_us / 1e3 / peak, 4)}
    d.update(extra)
    return d


def merged_inputs(lay, wl, device, step=0):
    """Packed rank-space q', k', v' of one new token, as a layer with merged weights would produce them: seeded
    N(0,1) draws in the IO dtype with zero padding lanes."""
    dt = synth.torch_dtype(wl.dtype)
    outs = []
    for tag, offs, ranks in (("Q", lay.offs_k, lay.r_k), ("K", lay.offs_k, lay.r_k), ("V", lay.offs_v, lay.r_v)):
        g = torch.Generator(device=device).manual_seed(synth.stream_seed(wl.index, "z_" + tag, extra=7000000 + step))
        x = torch.randn((wl.batch, 1, offs[-1]), generator=g, dtype=torch.float32, device=device)
        mask = torch.zeros(offs[-1], dtype=torch.bool, device=device)
        for h, r in enumerate(ranks):
            mask[offs[h]:offs[h] + r] = True
        outs.append((x * mask).to(dt).contiguous())
    return outs


def run_merged(args, wl):
    """The decode step as a layer with merged weights (Eq. 8) calls it: rank-space q', k', v' in, rank-space o' out.
    One JSON line: KV bytes per second against the HBM roofline, and parity of sampled units against the oracle,
    which receives the d_head-wide vectors whose projections are exactly those rank-space rows (x' U^T)."""
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    keep = [(0, 0), (wl.batch - 1, wl.n_heads - 1)]
    lay, ranks, U_k, U_v, hist, _, _, _ = build_layer(wl, device, binding, keep)
    n0 = wl.context
    qp, kp, vp = merged_inputs(lay, wl, device)
    outp = torch.empty((wl.batch, 1, lay.offs_v[-1]), dtype=qp.dtype, device=device)
    def step():
        lay.set_len(n0)
        lay.decode_step(qp, kp, vp, out=outp, q_preprojected=True, kv_preprojected=True, out_lowrank=True)
    steps, warmup = min(args.steps, 100), max(3, min(args.warmup, 10))
    sampler = ClockSampler(device.index or 0)
    sampler.start(); time.sleep(0.2)
    l0 = lay.launch_count()
    k_us, s_us = timed_kernel(lay, device, step, steps, warmup)
    launches = lay.launch_count() - l0
    clocks = sampler.stop()
    bytes_step = algorithmic_bytes(wl, ranks, ranks, n0 + 1)
    peak, peak_src = measured_peaks()
    from oracle import eigen_attention as orc
    ref = orc.LayerOracle(wl.batch, wl.n_heads, wl.d_head, U_k, U_v, tracked=keep)
    errs = []
    for (b, h) in keep:
        back = lambda x, offs, U: x[b, 0, offs[h]:offs[h] + U[h].shape[1]].double().cpu().numpy() @ U[h].astype(np.float64).T
        K = np.concatenate([hist[(b, h)][0], back(kp, lay.offs_k, U_k)[None]])
        V = np.concatenate([hist[(b, h)][1], back(vp, lay.offs_v, U_v)[None]])
        exp = orc.decode_head(back(qp, lay.offs_k, U_k), K, V, U_k[h], U_v[h], lowrank_out=True)
        got = outp[b, 0, lay.offs_v[h]:lay.offs_v[h] + ranks[h]].double().cpu().numpy()
        errs.append(float(np.abs(got - exp).max()))
    achieved = bytes_step / k_us / 1e3
    print(json.dumps({
        "metric": "rank-r decode attention KV GB/s, merged-weight call (rank-space q', k', v' in, o' out)",
        "value": bytes_step / s_us / 1e3, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warmup,
        "ms_per_step": s_us * 1e-3, "us_per_step": s_us, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 storage, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "n_heads": wl.n_heads, "rank": sorted(set(ranks)), "context": n0,
                   "flags": "EA_Q_PREPROJECTED | EA_KV_PREPROJECTED | EA_OUT_LOWRANK", "l2": "inputs larger than L2"},
        "roofline": {"bound": "hbm", "kernel": "decode_splitkv_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_src, "kernel_us": k_us, "algorithmic_bytes": bytes_step,
                     "traffic": None},
        "gpu_launches": launches, "clocks": clocks,
        "parity_sampled_units": {"units": len(errs), "max_abs": max(errs), "tolerance": "max_abs <= 2e-2"},
    }))


def workload_table(device, binding, lay2, wl2, ranks2, q2, k2, v2, steps=30, warmup=3):
    """The other workloads, each as one short timed region of the call a user makes: kernel time from the library's
    event pair (median), step time on the stream, algorithmic bytes of the rows (or codes) the step must read, and
    the fraction of the measured copy bandwidth.  `lay2` is the headline layer, already filled; the variants that
    share its cache (unequal lengths, rotary embedding, quantised copy) reuse it."""
    import dataclasses
    peak, _ = measured_peaks()
    table = {}
    n2 = wl2.context
    out2 = torch.empty_like(q2)

    # ---- unequal lengths on the headline cache: sequence b keeps (b + 1) / B of the context
    lens = [max(1, n2 * (b + 1) // wl2.batch) for b in range(wl2.batch)]
    lay2.set_lens(lens)
    k_us, s_us = timed_kernel(lay2, device, lambda: lay2.decode(q2, out=out2), steps, warmup)
    row_bytes = sum(2 * 2 * r for r in ranks2)
    table["ragged"] = table_entry("decode_splitkv_kernel", k_us, s_us, sum(lens) * row_bytes, peak,
                                  workload=wl2.name + " with lens[b] = context * (b + 1) / batch")
    lay2.set_len(n2)

    # ---- ALiBi bias on the headline cache
    lay2.set_alibi(synth.alibi_slopes(wl2.n_heads))
    def step_alibi():
        lay2.set_len(n2); lay2.decode_step(q2, k2, v2, out=out2)
    k_us, s_us = timed_kernel(lay2, device, step_alibi, steps, warmup)
    table["alibi"] = table_entry("decode_splitkv_kernel", k_us, s_us, algorithmic_bytes(wl2, ranks2, ranks2, n2 + 1), peak,
                                 workload=wl2.name + " with per-head ALiBi slopes")
    lay2.set_alibi(None)
    lay2.set_len(n2)

    # ---- RoPE variant of decode on the headline cache (full-rank query, keys lifted and rotated)
    lay2.set_rope(ROPE_BASE)
    def step_rope():
        lay2.set_len(n2); lay2.decode_step(q2, k2, v2, out=out2)
    k_us, s_us = timed_kernel(lay2, device, step_rope, steps, warmup)
    table["rope"] = table_entry("decode_rope_kernel", k_us, s_us, algorithmic_bytes(wl2, ranks2, ranks2, n2 + 1), peak,
                                workload=wl2.name + " with rotary position embedding")
    lay2.set_rope(0.0)
    lay2.set_len(n2)

    # ---- merged weights (Eq. 8): rank-space q', k', v' in, rank-space o' out; no multiplication by U in the step
    qp, kp, vp = merged_inputs(lay2, wl2, device)
    outp = torch.empty((wl2.batch, 1, lay2.offs_v[-1]), dtype=q2.dtype, device=device)
    def step_merged():
        lay2.set_len(n2)
        lay2.decode_step(qp, kp, vp, out=outp, q_preprojected=True, kv_preprojected=True, out_lowrank=True)
    k_us, s_us = timed_kernel(lay2, device, step_merged, steps, warmup)
    table["merged_weights"] = table_entry("decode_splitkv_kernel", k_us, s_us, algorithmic_bytes(wl2, ranks2, ranks2, n2 + 1), peak,
                                          workload=wl2.name + ", rank-space q', k', v' in and o' out")
    lay2.set_len(n2)

    # ---- quantised copies of the headline cache
    for bits, G in QUANT_LEGS:
        lay2.set_len(n2)
        lay2.quant_attach(bits, G)
        lay2.quant_sync()
        def step_quant():
            lay2.set_len(n2); lay2.append_kv(k2, v2); lay2.decode_quant(q2, out=out2)
        k_us, s_us = timed_kernel(lay2, device, step_quant, steps, warmup)
        nq = n2 // G * G
        codes = wl2.batch * (nq // G) * sum(lay2.quant_layout(h)[1] for h in range(wl2.n_heads))
        tail = wl2.batch * (n2 + 1 - nq) * row_bytes
        table[f"quant_{bits}bit_g{G}"] = table_entry("decode_quant_mma_kernel" if bits == 4 else "decode_quant_kernel", k_us, s_us, codes + tail, peak,
                                                     workload=wl2.name + f", {bits}-bit codes, group {G}",
                                                     bytes_16bit=algorithmic_bytes(wl2, ranks2, ranks2, n2 + 1))
        lay2.quant_detach()
    lay2.set_len(n2)
    return table


def workload_table_own_layers(device, binding, steps=30, warmup=3):
    """Workloads that need a layer of their own: the long-context layer (B = 1, 2), the batch x context sweep of the
    layer with per-head ranks, and the grouped-query layer."""
    import dataclasses
    peak, _ = measured_peaks()
    table = {}
    wl = synth.WORKLOADS["llama2_7b_b16_n32k"]             # the headline layer on a paged cache, pages of 128 rows
    lay, ranks, _, _, _, q, kn, vn = build_layer(wl, device, binding, page_rows=128)
    out = torch.empty_like(q)
    def step_paged():
        lay.set_len(wl.context); lay.decode_step(q, kn, vn, out=out)
    k_us, s_us = timed_kernel(lay, device, step_paged, steps, warmup)
    table["paged_cache"] = table_entry("decode_splitkv_kernel", k_us, s_us, algorithmic_bytes(wl, ranks, ranks, wl.context + 1), peak,
                                       workload=wl.name + ", page table with pages of 128 rows shuffled over the pool")
    lay.set_rope(10000.0)                                  # the same paged layer as a layer with rotary embedding
    k_us, s_us = timed_kernel(lay, device, step_paged, steps, warmup)
    table["paged_cache[rope]"] = table_entry("decode_rope_kernel", k_us, s_us, algorithmic_bytes(wl, ranks, ranks, wl.context + 1),
                                             peak, workload=wl.name + ", rotary embedding, pages of 128 rows shuffled over the pool")
    del lay
    torch.cuda.empty_cache()
    for b in (1, 2):
        wl = dataclasses.replace(synth.WORKLOADS["mpt_7b_long"], batch=b)
        lay, ranks, _, _, _, q, kn, vn = build_layer(wl, device, binding)
        out = torch.empty_like(q)
        def step():
            lay.set_len(wl.context); lay.decode_step(q, kn, vn, out=out)
        k_us, s_us = timed_kernel(lay, device, step, steps, warmup)
        table[f"mpt_7b_long[batch={b}]"] = table_entry("decode_splitkv_kernel", k_us, s_us,
                                                       algorithmic_bytes(wl, ranks, ranks, wl.context + 1), peak)
        del lay
        torch.cuda.empty_cache()
    for b in (1, 4, 16, 64):
        wl = dataclasses.replace(synth.WORKLOADS["opt_6p7b_hetero"], batch=b, context=32768)
        lay, ranks, _, _, _, q, kn, vn = build_layer(wl, device, binding)
        out = torch.empty_like(q)
        for n in (2048, 8192, 32768):                       # the rows beyond n stay in the cache and are not read
            def step():
                lay.set_len(n); lay.decode_step(q, kn, vn, out=out)
            k_us, s_us = timed_kernel(lay, device, step, steps, warmup)
            wn = dataclasses.replace(wl, context=n)
            table[f"opt_6p7b_hetero[batch={b},context={n}]"] = table_entry(
                "decode_splitkv_kernel", k_us, s_us, algorithmic_bytes(wn, ranks, ranks, n + 1), peak,
                l2="cache-resident" if algorithmic_bytes(wn, ranks, ranks, n + 1) < 126e6 else "larger than L2")
        del lay
        torch.cuda.empty_cache()
    wl = synth.WORKLOADS["llama3_8b_gqa_b16_n32k"]
    g = synth.GQA_GROUP[wl.name]
    lay, ranks, _, _, _, _, kn, vn = build_layer(wl, device, binding)
    q = synth.gaussian_query(wl.batch, wl.n_heads * g, wl.d_head, wl.q_scale, wl.index, dtype=synth.torch_dtype(wl.dtype), device=device)
    out = torch.empty_like(q)
    def step_gqa():
        lay.set_len(wl.context); lay.append_kv(kn, vn); lay.decode_gqa(q, g, out=out)
    k_us, s_us = timed_kernel(lay, device, step_gqa, steps, warmup)
    table[wl.name] = table_entry("decode_gqa_mma_kernel", k_us, s_us, algorithmic_bytes(wl, ranks, ranks, wl.context + 1), peak,
                                 group=g)
    # the same layer with the rotary embedding these models use (the bytes counted are the rows of the cache, read once)
    lay.set_rope(10000.0)
    k_us, s_us = timed_kernel(lay, device, step_gqa, steps, warmup)
    table[wl.name + "[rope]"] = table_entry("decode_gqa_rope_kernel", k_us, s_us,
                                            algorithmic_bytes(wl, ranks, ranks, wl.context + 1), peak, group=g, rope=True)
    del lay
    torch.cuda.empty_cache()
    return table


def prefill_measure(wl, device, steps, warmup, impl=0, rope=False):
    """Times eigen_attn_prefill on the prompt workload; returns a small dict (call time, attention-kernel time,
    TFLOP/s of the causal contractions, fraction of the measured bf16 peak)."""
    from paper_2408_05646_b200 import binding
    ranks = synth.draw_ranks(wl.n_heads, wl.ranks, wl.index)
    U_k = synth.make_bases(wl.d_head, ranks, wl.index, "U_K")
    U_v = synth.make_bases(wl.d_head, ranks, wl.index, "U_V")
    dt = synth.torch_dtype(wl.dtype)
    T = wl.context
    lay = binding.EigenAttnLayer(wl.batch, wl.n_heads, wl.d_head, T + 1, dt, U_k, U_v, max_prefill_tokens=T, device=device,
                                 rope_prompt_scratch=rope)
    if rope:                                       # Section 4.3: full-rank rotated queries against lifted, rotated keys
        lay.set_rope(10000.0)
    if impl:
        lay.set_option(binding.EA_OPT_PREFILL_IMPL, impl)
    W = {t: synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_" + t, device=device) for t in "KVQ"}
    k = synth.lowrank_rows(W["K"], wl.batch, T, wl.sigma, wl.index, "K", dtype=dt, device=device)
    v = synth.lowrank_rows(W["V"], wl.batch, T, wl.sigma, wl.index, "V", dtype=dt, device=device)
    q = synth.lowrank_rows(W["Q"], wl.batch, T, wl.sigma, wl.index, "Q", dtype=dt, device=device)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream(device)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        a.record(stream); b.record(stream)
    for _ in range(warmup):
        lay.set_len(0); lay.prefill(q, k, v, out=out)
    torch.cuda.synchronize(device)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for i in range(steps):
        lay.set_decode_events(ev[i][0], ev[i][1])
        lay.set_len(0); lay.prefill(q, k, v, out=out)
    t1.record(stream)
    torch.cuda.synchronize(device)
    lay.set_decode_events(None, None)
    lay.poll_status()
    ms = t0.elapsed_time(t1) / steps
    kern = sum(a.elapsed_time(b) for a, b in ev) / steps
    # causal contractions: Q'K'^T over r_k (d_head wide with the rotary embedding) and PV' over r_v
    flop = 2 * (wl.batch * T * (T + 1) // 2) * sum((wl.d_head if rope else r) + r for r in ranks)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["bf16_tflops"]) if os.path.exists(peaks_path) else 1590.0
    tf = flop / (kern * 1e-3) / 1e12
    # the projection kernel (HBM-bound): q, k, v in, cache rows and Q' out, against the measured copy bandwidth
    es = 2 if wl.dtype == "bf16" else 4
    proj_bytes = wl.batch * T * (3 * wl.n_heads * wl.d_head + sum(3 * r for r in ranks)) * es
    proj_ms = ms - kern
    hbm, _ = measured_peaks()
    return {"workload": wl.name, "ms_per_call": ms, "attention_kernel_ms": kern, "attention_tflops": tf,
            "projection_ms": proj_ms, "projection_gbs": proj_bytes / (proj_ms * 1e-3) / 1e9,
            "projection_frac_of_hbm": proj_bytes / (proj_ms * 1e-3) / 1e9 / hbm,
            "bound": "tensor", "peak_tflops": peak, "frac": tf / peak,
            "peak_source": "measured burst" if os.path.exists(peaks_path) else "fallback",
            "flop_counted": "causal Q'K'^T + PV' (projections and lift excluded)"}


def run_prefill(args, wl):
    """Causal rank-r prefill of the whole prompt (project K/V and write the cache, project Q, attention on the
    tensor cores, lift): one JSON line with time, TFLOP/s of the causal contractions and the tensor roofline."""
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    ranks = synth.draw_ranks(wl.n_heads, wl.ranks, wl.index)
    U_k = synth.make_bases(wl.d_head, ranks, wl.index, "U_K")
    U_v = synth.make_bases(wl.d_head, ranks, wl.index, "U_V")
    dt = synth.torch_dtype(wl.dtype)
    T = wl.context
    lay = binding.EigenAttnLayer(wl.batch, wl.n_heads, wl.d_head, T + 1, dt, U_k, U_v, max_prefill_tokens=T, device=device,
                                 rope_prompt_scratch=args.rope)
    if args.rope:                                  # Section 4.3: rotated full-rank queries against lifted, rotated keys
        lay.set_rope(10000.0)
    if args.prefill_impl:
        lay.set_option(binding.EA_OPT_PREFILL_IMPL, args.prefill_impl)
    W = {t: synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_" + t, device=device) for t in "KVQ"}
    k = synth.lowrank_rows(W["K"], wl.batch, T, wl.sigma, wl.index, "K", dtype=dt, device=device)
    v = synth.lowrank_rows(W["V"], wl.batch, T, wl.sigma, wl.index, "V", dtype=dt, device=device)
    q = synth.lowrank_rows(W["Q"], wl.batch, T, wl.sigma, wl.index, "Q", dtype=dt, device=device)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream(device)
    steps, warmup = min(args.steps, 20), min(args.warmup, 5)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        a.record(stream); b.record(stream)
    for _ in range(warmup):
        lay.set_len(0); lay.prefill(q, k, v, out=out)
    torch.cuda.synchronize(device)
    sampler = ClockSampler(device.index or 0)
    sampler.start(); time.sleep(0.2)
    l0 = lay.launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for i in range(steps):
        lay.set_decode_events(ev[i][0], ev[i][1])
        lay.set_len(0); lay.prefill(q, k, v, out=out)
    t1.record(stream)
    torch.cuda.synchronize(device)
    lay.set_decode_events(None, None)
    clocks = sampler.stop()
    lay.poll_status()
    ms = t0.elapsed_time(t1) / steps
    kern = sum(a.elapsed_time(b) for a, b in ev) / steps
    pairs = wl.batch * T * (T + 1) // 2                       # causal (query, key) pairs per head, summed over the batch
    # Q'K'^T and PV' over the lower triangle (with the rotary embedding the score product is d_head wide)
    flop = 2 * pairs * sum((wl.d_head if args.rope else r) + r for r in ranks)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak, src = 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"
    if os.path.exists(peaks_path):
        peak, src = float(json.load(open(peaks_path))["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
    # parity of sampled rows of two units against the oracle (one by one)
    from oracle import eigen_attention as orc
    errs = []
    for (b, h) in [(0, 0), (wl.batch - 1, wl.n_heads - 1)]:
        rows = [0, 1, 127, 128, 1000, T - 1]
        kk, vv = k[b, :, h].double().cpu().numpy(), v[b, :, h].double().cpu().numpy()
        for t in rows:
            qt = q[b, t, h].double().cpu().numpy()
            if args.rope:                          # row t of the prompt form = the generation form over rows 0..t
                ref = orc.decode_head_rope(qt, kk[:t + 1] @ U_k[h].astype(np.float64), vv[:t + 1] @ U_v[h].astype(np.float64),
                                           U_k[h], U_v[h], 10000.0, False)
            else:
                ref = orc.decode_head(qt, kk[:t + 1], vv[:t + 1], U_k[h], U_v[h])
            errs.append(float(np.abs(out[b, t, h].double().cpu().numpy() - ref).max()))
    achieved = flop / (kern * 1e-3) / 1e12
    print(json.dumps({
        "metric": "causal rank-r prefill attention TFLOP/s (B=4, T=4096, 7B layer)" + (", rotary embedding" if args.rope else ""),
        "value": flop / (ms * 1e-3) / 1e12,
        "unit": "TFLOP/s", "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 operands, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "n_heads": wl.n_heads, "d_head": wl.d_head, "rank": sorted(set(ranks)),
                   "prompt": T, "flop_counted": "2*pairs*(r_k+r_v) over the causal triangle; projections and lift excluded"},
        "roofline": {"bound": "tensor", "kernel": "prefill attention kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "peak_source": src, "kernel_ms": kern, "traffic": None},
        "gpu_launches": lay.launch_count() - l0, "clocks": clocks,
        "parity_sampled_rows": {"rows": len(errs), "max_abs": max(errs), "tolerance": "max_abs <= 2e-2"},
    }))


def run_ragged(args, wl):
    """Decode over a batch whose sequences differ in length (eigen_attn_set_lens): sequence b keeps
    (b + 1) / B of the context.  One JSON line: KV bytes of the TRUE lengths per second against the HBM roofline,
    and the same batch with every sequence at full length beside it."""
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    lay, ranks, U_k, U_v, _, q, k_new, v_new = build_layer(wl, device, binding)
    n0, Bn = wl.context, wl.batch
    lens = [max(1, n0 * (b + 1) // Bn) for b in range(Bn)]
    stream = torch.cuda.current_stream(device)
    out = torch.empty_like(q)
    steps, warmup = args.steps, max(args.warmup, 3)

    def timed(prepare):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            a.record(stream); b.record(stream)
        prepare()
        for _ in range(warmup):
            lay.decode(q, out=out)
        torch.cuda.synchronize(device)
        for i in range(steps):
            lay.set_decode_events(ev[i][0], ev[i][1])
            lay.decode(q, out=out)
        torch.cuda.synchronize(device)
        lay.set_decode_events(None, None)
        return sum(a.elapsed_time(b) for a, b in ev) / steps * 1e3      # us per decode kernel

    sampler = ClockSampler(device.index or 0)
    sampler.start(); time.sleep(0.2)
    l0 = lay.launch_count()
    us_ragged = timed(lambda: lay.set_lens(lens))
    launches = lay.launch_count() - l0
    us_full = timed(lambda: lay.set_len(n0))
    clocks = sampler.stop()
    lay.poll_status()
    row_bytes = sum(2 * (rk + rv) for rk, rv in zip(ranks, ranks))          # bf16 K' + V' row of all heads
    bytes_true = sum(lens) * row_bytes
    peak, src = measured_peaks()
    achieved = bytes_true / (us_ragged * 1e-6) / 1e9
    print(json.dumps({
        "metric": "rank-r decode attention KV GB/s, batch of unequal lengths", "value": achieved, "unit": "GB/s",
        "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": us_ragged * 1e-3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 storage, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl.name + " with lens[b] = context * (b + 1) / batch", "batch": Bn, "context": n0,
                   "mean_len": sum(lens) / Bn, "l2": "inputs larger than L2"},
        "roofline": {"bound": "hbm", "kernel": "decode_splitkv_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": src, "kernel_us": us_ragged, "algorithmic_bytes": bytes_true,
                     "traffic": None},
        "all_sequences_at_full_length": {"kernel_us": us_full, "GB/s": Bn * n0 * row_bytes / (us_full * 1e-6) / 1e9},
        "gpu_launches": launches, "clocks": clocks,
    }))


def run_gqa(args, wl):
    """Grouped-query decode step: append the new token's K/V rows, then one pass over the rank-r cache of every K/V
    head serves its whole group of query heads.  One JSON line: KV GB/s of that pass against the HBM roofline, and
    the same step for the query heads one by one through the multi-head kernel for comparison."""
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    g = synth.GQA_GROUP[wl.name.split("[")[0]]
    keep = [0, wl.n_heads - 1]
    lay, ranks, U_k, U_v, hist, _, k_new, v_new = build_layer(wl, device, binding, [(0, h) for h in keep])
    dt = synth.torch_dtype(wl.dtype)
    q = synth.gaussian_query(wl.batch, wl.n_heads * g, wl.d_head, wl.q_scale, wl.index, dtype=dt, device=device)
    out = torch.empty_like(q)
    n0 = wl.context
    stream = torch.cuda.current_stream(device)
    steps, warmup = min(args.steps, 100), max(3, min(args.warmup, 10))
    rope = {"base": 10000.0, "interleaved": False} if args.rope else None
    if rope:                                       # Section 4.3 for the group: the form the Llama-3 models run
        lay.set_rope(rope["base"])
    lay.set_option(binding.EA_OPT_GQA_IMPL, args.gqa_impl)
    gqa_kernel = "decode_gqa_rope_kernel" if rope else "decode_gqa_kernel" if args.gqa_impl == 1 else "decode_gqa_mma_kernel"

    def step():
        lay.set_len(n0)
        lay.append_kv(k_new, v_new)
        lay.decode_gqa(q, g, out=out)

    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, c in ev:
        a.record(stream); c.record(stream)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize(device)
    sampler = ClockSampler(device.index or 0)
    sampler.start(); time.sleep(0.2)
    l0 = lay.launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for i in range(steps):
        lay.set_decode_events(ev[i][0], ev[i][1])
        step()
    t1.record(stream)
    torch.cuda.synchronize(device)
    lay.set_decode_events(None, None)
    clocks = sampler.stop()
    launches = lay.launch_count() - l0
    lay.poll_status()
    ms = t0.elapsed_time(t1) / steps
    kern = sum(a.elapsed_time(c) for a, c in ev) / steps
    bytes_step = algorithmic_bytes(wl, ranks, ranks, n0 + 1)
    peak, peak_src = measured_peaks()
    # the same query heads one group member at a time through the multi-head decode kernel (g passes over the cache)
    q_one = [q[:, :, i::g].contiguous() for i in range(g)]
    o_one = torch.empty_like(q_one[0])
    for _ in range(3):
        for i in range(g):
            lay.decode(q_one[i], out=o_one)
    torch.cuda.synchronize(device)
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    for _ in range(10):
        for i in range(g):
            lay.decode(q_one[i], out=o_one)
    a1.record(stream)
    torch.cuda.synchronize(device)
    ms_one_by_one = a0.elapsed_time(a1) / 10
    # parity of the sampled units against the oracle
    from oracle import eigen_attention as orc
    ref = orc.LayerOracle(wl.batch, wl.n_heads, wl.d_head, U_k, U_v, tracked=[(0, h) for h in keep], rope=rope)
    for h in keep:
        ref.append_unit_rows((0, h), hist[(0, h)][0], hist[(0, h)][1])
    ref.set_len(n0)
    ref.append_kv(k_new.double().cpu().numpy(), v_new.double().cpu().numpy())
    exp = ref.decode_gqa(q.double().cpu().numpy(), g)
    got = out.double().cpu().numpy()
    errs = [float(np.abs(got[0, 0, h * g + i] - exp[0, 0, h * g + i]).max()) for h in keep for i in range(g)]
    achieved = bytes_step / (kern * 1e-3) / 1e9
    print(json.dumps({
        "metric": "grouped-query rank-r decode KV GB/s (B=16, n=32k, 8 K/V heads x 4 query heads)" + (", rotary embedding" if rope else ""),
        "value": bytes_step / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warmup,
        "ms_per_step": ms, "us_per_step": ms * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 storage and operands, f32 accumulate", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "kv_heads": wl.n_heads, "group": g, "d_head": wl.d_head,
                   "rank": sorted(set(ranks)), "context": n0, "new_tokens": 1, "cache_gb": bytes_step / 1e9,
                   "l2": "inputs larger than L2: every step streams the whole rank-r cache"},
        "roofline": {"bound": "hbm", "kernel": gqa_kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_src, "kernel_us": kern * 1e3,
                     "algorithmic_bytes": bytes_step, "traffic": None},
        "one_query_head_at_a_time_us": ms_one_by_one * 1e3,
        "gpu_launches": launches, "clocks": clocks,
        "parity_sampled_units": {"query_heads": len(errs), "max_abs": max(errs), "tolerance": "max_abs <= 2e-2"},
    }))


def run_quant(args, wl):
    """Decode step over the quantised rank-r cache (4-bit codes, group --quant): append the new token's 16-bit rows,
    then one pass over the codes.  One JSON line: bytes of codes and scales read per second against the HBM
    roofline, the 16-bit decode of the same cache beside it, and parity of sampled units against the oracle."""
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    G = args.quant
    keep = [0, wl.n_heads - 1]
    lay, ranks, U_k, U_v, hist, q, k_new, v_new = build_layer(wl, device, binding, [(0, h) for h in keep])
    lay.quant_attach(4, G)
    lay.quant_sync()
    n0 = wl.context
    nq = n0 // G * G
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream(device)
    steps, warmup = min(args.steps, 100), max(3, min(args.warmup, 10))

    def step():
        lay.set_len(n0)
        lay.append_kv(k_new, v_new)
        lay.decode_quant(q, out=out)

    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, c in ev:
        a.record(stream); c.record(stream)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize(device)
    sampler = ClockSampler(device.index or 0)
    sampler.start(); time.sleep(0.2)
    l0 = lay.launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for i in range(steps):
        lay.set_decode_events(ev[i][0], ev[i][1])
        step()
    t1.record(stream)
    torch.cuda.synchronize(device)
    lay.set_decode_events(None, None)
    clocks = sampler.stop()
    launches = lay.launch_count() - l0
    lay.poll_status()
    ms = t0.elapsed_time(t1) / steps
    kern = sum(a.elapsed_time(c) for a, c in ev) / steps
    # bytes one step must read: every block of codes and scales, plus the 16-bit rows not quantised yet
    block_bytes = [lay.quant_layout(h)[1] for h in range(wl.n_heads)]
    bytes_codes = wl.batch * (nq // G) * sum(block_bytes)
    bytes_tail = wl.batch * (n0 + 1 - nq) * 2 * sum(ranks) * 2
    bytes_step = bytes_codes + bytes_tail
    bytes_16bit = algorithmic_bytes(wl, ranks, ranks, n0 + 1)
    peak, peak_src = measured_peaks()
    # the 16-bit decode of the same cache
    for _ in range(3):
        lay.decode(q, out=out)
    torch.cuda.synchronize(device)
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    for _ in range(20):
        lay.decode(q, out=out)
    a1.record(stream)
    torch.cuda.synchronize(device)
    ms_16bit = a0.elapsed_time(a1) / 20
    step()
    torch.cuda.synchronize(device)
    # parity of the sampled units: the oracle keeps 16-bit rows (Section 2, p = 16) and quantises those
    from oracle import eigen_attention as orc
    dt = synth.torch_dtype(wl.dtype)
    storage = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dt).double().numpy()
    ref = orc.LayerOracle(wl.batch, wl.n_heads, wl.d_head, U_k, U_v, tracked=[(0, h) for h in keep], storage=storage)
    for h in keep:
        ref.append_unit_rows((0, h), hist[(0, h)][0], hist[(0, h)][1])
    ref.set_len(n0)
    ref.append_kv(k_new.double().cpu().numpy(), v_new.double().cpu().numpy())
    exp = ref.decode_quant(q.double().cpu().numpy(), 4, G)
    got = out.double().cpu().numpy()
    errs = [float(np.abs(got[0, 0, h] - exp[(0, h)]).max()) for h in keep]
    achieved = bytes_step / (kern * 1e-3) / 1e9
    print(json.dumps({
        "metric": "rank-r decode over the 4-bit cache, bytes of codes and scales read per second",
        "value": bytes_step / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warmup,
        "ms_per_step": ms, "us_per_step": ms * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "4-bit codes + f16 scales, f32 arithmetic", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "n_heads": wl.n_heads, "d_head": wl.d_head,
                   "rank": sorted(set(ranks)), "context": n0, "new_tokens": 1, "bits": 4, "group": G,
                   "quantised_rows": nq, "cache_gb": bytes_step / 1e9, "cache_gb_16bit": bytes_16bit / 1e9,
                   "l2": "inputs larger than L2: every step streams all codes"},
        "roofline": {"bound": "hbm", "kernel": "decode_quant_mma_kernel (+ combine)", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src, "kernel_us": kern * 1e3,
                     "algorithmic_bytes": bytes_step, "traffic": None},
        "decode_16bit_us": ms_16bit * 1e3, "speedup_over_16bit": ms_16bit / (kern if kern > 0 else ms),
        "gpu_launches": launches, "clocks": clocks,
        "parity_sampled_units": {"units": len(errs), "max_abs": max(errs), "tolerance": "max_abs <= 2e-2"},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b_b16_n32k", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--alibi", action="store_true", help="decode workloads: add the per-head ALiBi position bias")
    ap.add_argument("--rope", action="store_true", help="decode workloads: the RoPE variant (full-rank query, lifted rotated keys)")
    ap.add_argument("--quant", type=int, default=0, metavar="G",
                    help="decode workloads: attend over the 4-bit quantised cache with group size G (16, 32, 64, 128)")
    ap.add_argument("--merged", action="store_true", help="decode workloads: the step as a layer with merged weights calls it")
    ap.add_argument("--ragged", action="store_true", help="decode workloads: sequence b keeps (b + 1) / batch of the context")
    ap.add_argument("--no-prefill", action="store_true", help="skip the short prefill measurement in the decode line")
    ap.add_argument("--no-workloads", action="store_true", help="skip the table of the other workloads in the headline line")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (scaled-down profiling case)")
    ap.add_argument("--context", type=int, default=0, help="override the workload's context length")
    ap.add_argument("--prefill-impl", type=int, default=0, help="prefill workload: 0 auto, 1 CUDA-core, 2 tcgen05 kernel")
    ap.add_argument("--gqa-impl", type=int, default=0, choices=[0, 1],
                    help="grouped-query workload: 0 auto (warp-level products), 1 the tcgen05 kernel")
    args = ap.parse_args()
    VARIANT["alibi"] = bool(args.alibi)
    VARIANT["rope"] = bool(args.rope)
    if args.warmup < 3:
        args.warmup = 3
    wl = synth.WORKLOADS[args.workload]
    if args.batch or args.context:
        import dataclasses
        wl = dataclasses.replace(wl, batch=args.batch or wl.batch, context=args.context or wl.context,
                                 name=f"{wl.name}[batch={args.batch or wl.batch},context={args.context or wl.context}]")
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args, wl)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world:
        raise SystemExit(f"bench.py --gpus {args.gpus} must run as {args.gpus} rank(s), one per GPU, but WORLD_SIZE is "
                         f"{world}: launch it with `python -m torch.distributed.run --nnodes=1 --nproc-per-node {args.gpus} "
                         f"--master-addr 127.0.0.1 --master-port <port> bench.py --gpus {args.gpus} ...`")
    if args.workload in synth.GQA_GROUP:
        return run_gqa(args, wl)
    if args.quant:
        return run_quant(args, wl)
    if args.ragged:
        return run_ragged(args, wl)
    if args.merged:
        return run_merged(args, wl)
    if wl.name.startswith("prefill"):
        run_prefill(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
