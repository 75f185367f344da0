#!/usr/bin/env python
"""Benchmark of the NuPS sparse access path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload ...]

Default workload: the parameter-server microbenchmark.  A store of 100M keys x 128 fp32 (51.2 GB), batches of
1M keys ~ Zipf(1.0), the 1,000 most frequent keys replicated over 8 workers, replicas merged every 16 batches,
fast (atomic) mode.  One step = one pull of 1M keys + one push of 1M keys (+ the replica merge when it is due) +
PrepareSample and PullSample (keys and rows) of 1M keys from a Zipf(1.0) target over the whole store under pooled
reuse (BOUNDED, U = 16, G = 250).  Metric: key accesses per second (every pulled, pushed or sampled key is one).
The same run adds a `sweep` of the other points of that benchmark (skew 0 / 0.6 / 1.0 / 1.4, top-k 0 / 1k / 100k,
merge interval 1 / 16 / 256, the four sampling schemes) and one entry for each workload step (skip-gram, ComplEx,
matrix factorization).

With N > 1 every rank runs an independent replica of the workload on its own GPU (the path has no exchange step
on one node); the aggregate is total accesses over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2104_00501_b200 import inputs  # noqa: E402

VOCAB, DIM, BATCH, NEG, WINDOW = 1_000_000, 300, 4096, 3, 5
U_REUSE, G_POOL, SYNC_EVERY, WORKERS, LR = 16, 250, 16, 8, 0.001
HOT_FRACTION = 0.01
TOKENS = 100_000_000
ACCESSES_PER_PAIR = 2 + NEG + (NEG + 2)          # direct pulls + sampled pulls + pushes
UPDATES_PER_PAIR = NEG + 2
MAX_DISTINCT_BATCHES = 4096
WORKLOAD_SGNS = ("SGNS word vectors: vocab 1M, dim 300, 100M-token Zipf(1.0) stream, window 5, 3 negatives unigram^0.75 "
                 "BOUNDED(U=16,G=250), batch 4096 pairs, top 1% keys replicated, sync every 16 batches, fast (atomic) mode")

# the parameter-server microbenchmark (the default line)
PS_KEYS, PS_LEN, PS_BATCH = 100_000_000, 128, 1 << 20
PS_SKEW, PS_TOPK, PS_SYNC, PS_LEVEL = 1.0, 1000, 16, "BOUNDED"
PS_SKEWS, PS_TOPKS, PS_SYNCS = (0.0, 0.6, 1.0, 1.4), (0, 1000, 100_000), (1, 16, 256)
PS_LEVELS = ("CONFORM", "BOUNDED", "LONG-TERM", "NON-CONFORM")
PS_KERNEL_EVENTS_EVERY = 4                      # repetitions of the timed region between two with kernel event pairs
PS_ORACLE_KEYS = 4_000_000                     # the oracle's table is scaled down to fit host memory everywhere
WORKLOAD_PS = ("PS microbenchmark: 100M keys x 128 fp32, 1M-key batches ~ Zipf(1.0), pull:push 1:1, top-1k keys replicated "
               "over 8 workers, replicas merged every 16 batches, plus PrepareSample+PullSample of 1M keys from a Zipf(1.0) "
               "target under BOUNDED(U=16,G=250); one step = one pull + one push + one sample pull, fast (atomic) mode")

# DRAM traffic of one launch of the fused step kernel (sgns_runs_kernel, 16 steps per launch, 10M-token stream), from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum); valid only for the kernel source it was captured on (sgns_kernel_sha1).
NCU_TRAFFIC = {"bytes_per_launch": 38886656 + 4509952, "sgns_kernel_sha1": "a667c3d0875db94740ac74690bf25a99019ad7aa"}

# The same for the kernels of the default line.  A 100M-key launch is too large to capture under ncu, so each figure comes
# from one capture of the same command with --ps-keys 4000000 (2 GB table, the same 1M-key batches, kernels and launch shapes;
# see profiles/ps_line_kernels_dram_traffic.md): DRAM bytes of that launch, its algorithmic bytes, and the hash of the
# kernel's source text at the time.  The traffic reported for the timed launch is scaled by the algorithmic bytes, which is
# what the capture shows the traffic follows.  A kernel whose source has changed since reports no traffic.
NCU_TRAFFIC_PS = {
    "pull": {"dram_bytes": 216757504 + 481016320, "algorithmic_bytes": 694418688, "sha1": "d6be6ab4363bba8db6eba30551f6fe4750727ba0"},
    "push": {"dram_bytes": 712619776 + 126636032, "algorithmic_bytes": 847772160, "sha1": "0a8c080becb64f3aaf867fbcd3f9c9bc21bc1399"},
    "sample_rows": {"dram_bytes": 27681024 + 478645504, "algorithmic_bytes": 562094080,
                    "sha1": "d6be6ab4363bba8db6eba30551f6fe4750727ba0"},
}
PS_KERNEL_SOURCE = {   # kind -> (kernel name, start and end markers of its source text in store.cu)
    "pull": ("gather8_kernel", "// The same gather with 256-bit loads and stores", "nups_status nups_gather_internal("),
    "push": ("push_atomic_kernel", "// push, fast mode: 128-bit reductions", "// push, deterministic mode"),
    "sample_rows": ("gather8_kernel", "// The same gather with 256-bit loads and stores", "nups_status nups_gather_internal("),
}


def kernel_source_sha1(start_marker, end_marker, name="store.cu"):
    """Hash of a kernel's source text (the part of the file between two markers)."""
    src = open(os.path.join(ROOT, "paper_2104_00501_b200", "csrc", name)).read()
    a = src.index(start_marker)
    return hashlib.sha1(src[a:src.index(end_marker, a)].encode()).hexdigest()


def sgns_kernel_sha1():
    """Hash of the fused skip-gram kernel's source text (the part of steps.cu between its heading comment and the next
    kernel's): the ncu traffic figure below is only reported for the source it was captured on."""
    src = open(os.path.join(ROOT, "paper_2104_00501_b200", "csrc", "steps.cu")).read()
    a = src.index("// skip-gram with negative sampling.  One warp works on one pair at a time")
    b = src.index("// ComplEx with AdaGrad.")
    return hashlib.sha1(src[a:b].encode()).hexdigest()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for n, v in zip(names, r[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# workload construction (seeded, synthetic; stands in for the One Billion Word Benchmark)
# --------------------------------------------------------------------------------------------
def make_sgns_data(device, n_batches, seed=0, store=None):
    """Token stream in chunks: word counts, the pairs of the first batches, integer sampling weights.
    With a store, every token is also counted as an access to its input key and to its output key."""
    cdf = inputs.zipf_cdf(VOCAB, 1.0, device)
    counts = torch.zeros(VOCAB, dtype=torch.int64, device=device)
    chunk = 10_000_000
    first = None
    for i in range(TOKENS // chunk):
        t = inputs.zipf_keys(chunk, VOCAB, 1.0, seed * 1000 + i, device, cdf=cdf)
        counts += torch.bincount(t, minlength=VOCAB)
        if store is not None:
            t32 = t.to(torch.int32)
            store.count_accesses(t32)
            store.count_accesses(t32 + VOCAB)
        if i == 0:
            first = t
    need = n_batches * BATCH
    tok = first[: need // (2 * WINDOW) + 4 * WINDOW]
    c, o = inputs.skipgram_pairs(tok, WINDOW)
    assert c.numel() >= need, "token prefix too short for the requested number of batches"
    c, o = c[:need].to(torch.int32).contiguous(), (o[:need] + VOCAB).to(torch.int32).contiguous()
    weights = inputs.integer_weights(counts).to(torch.int32)
    return c, o, counts, weights


def build_store(binding, device, n_batches, seed, deterministic=False, sync_interval=SYNC_EVERY, clip_factor=0.0):
    s = binding.Store(2 * VOCAB, DIM, workers=WORKERS, sync_interval=sync_interval, deterministic=deterministic,
                      track_ownership=False, clip_factor=clip_factor)
    s.init_uniform(0, 1, 0.5 / DIM)
    c, o, counts, weights = make_sgns_data(device, n_batches, seed, store=s)
    hot = s.select_hot(True, int(HOT_FRACTION * 2 * VOCAB))          # the most frequently accessed 1 % of keys
    if hot.numel():
        s.set_management(hot, binding.REPLICATE)
    dist = s.register_distribution(VOCAB, weights.contiguous(), VOCAB, binding.BOUNDED, U=U_REUSE, G=G_POOL, seed=7)
    return s, dist, hot.long(), c, o, weights


def max_over_ranks(values, world, device):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank's time counts)."""
    if world <= 1:
        return [float(x) for x in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_throughput(units_per_rank, seconds, world):
    """Whole-job throughput of `world` independent replicas: all units over the slowest rank's time."""
    return units_per_rank * world / seconds


def run_sgns_line(args, rank, world, device):
    from paper_2104_00501_b200 import binding
    hbm_peak, peak_kind = peaks()
    nb = min(-(-(args.steps + args.warmup) // 64) * 64, MAX_DISTINCT_BATCHES)
    s, dist, hot, c, o, weights = build_store(binding, device, nb, seed=rank)
    loss = torch.zeros(1, dtype=torch.float32, device=device)

    def batch(i):
        j = (i % nb) * BATCH
        return c[j:j + BATCH], o[j:j + BATCH]

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    # the timed loop hands the library CHUNK consecutive batches per call (nups_run_sgns): every batch is still one
    # step of the path, but the steps between two replica merges share a kernel launch
    CHUNK = 4 * SYNC_EVERY
    assert nb % CHUNK == 0 or nb < CHUNK
    losses = torch.zeros(CHUNK, dtype=torch.float32, device=device)

    def run(first, count):
        done = 0
        while done < count:
            j = (first + done) % nb
            m = min(CHUNK, count - done, nb - j)
            s.run_sgns(c[j * BATCH:(j + m) * BATCH], o[j * BATCH:(j + m) * BATCH], BATCH, dist, NEG, LR, losses[:m])
            done += m
        return m

    run(0, args.warmup)
    launches0 = s.stats()["launches"]
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with ClockSampler(torch.cuda.current_device()) as clk:
        ev0.record()
        last = run(args.warmup, args.steps)
        ev1.record()
        barrier()
    loss.copy_(losses[:last].mean().reshape(1))          # mean loss over the last call's steps
    ms = ev0.elapsed_time(ev1)
    launches = s.stats()["launches"] - launches0
    final_loss = float(loss.item())

    # end to end through the public API (`Store.run_sgns`, CHUNK steps per call, as in the device-timed loop): every
    # step's pairs start in pinned host memory and are copied to the device inside the timed region, every step's
    # loss is copied back and read by the host.  Two buffers in flight: the host waits for call k-1's losses to
    # have landed before it issues call k+1.
    n_chunks = nb // CHUNK if nb >= CHUNK else 0
    e2e_steps = min(args.steps, nb) // CHUNK * CHUNK if n_chunks else 0
    e2e_s = float("nan")
    if e2e_steps:
        hchunks = torch.stack([c.view(n_chunks, CHUNK * BATCH), o.view(n_chunks, CHUNK * BATCH)], dim=1).cpu().pin_memory()
        dbuf = [torch.empty(2, CHUNK * BATCH, dtype=torch.int32, device=device) for _ in range(2)]
        dls = [torch.zeros(CHUNK, device=device) for _ in range(2)]
        hls = [torch.zeros(CHUNK, dtype=torch.float32).pin_memory() for _ in range(2)]
        done = [torch.cuda.Event(), torch.cuda.Event()]
        seen = 0.0
        barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps // CHUNK):
            k = i & 1
            if i >= 2:
                done[k].synchronize()
                seen += float(hls[k].sum())                   # the host really reads every step's loss
            dbuf[k].copy_(hchunks[i % n_chunks], non_blocking=True)
            s.run_sgns(dbuf[k][0], dbuf[k][1], BATCH, dist, NEG, LR, dls[k])
            hls[k].copy_(dls[k], non_blocking=True)
            done[k].record()
        for k in range(2):
            done[k].synchronize()
            seen += float(hls[k].sum())
        barrier()
        e2e_s = time.perf_counter() - t0
        assert np.isfinite(seen)

    # the same with one library call per step (`Store.step_sgns`): what a caller pays who needs every step's loss
    # before it decides on the next step
    hpairs = torch.stack([c.view(nb, BATCH), o.view(nb, BATCH)], dim=1).cpu().pin_memory()      # [nb, 2, BATCH]
    step_calls = min(args.steps, 2048)
    dpairs2 = [torch.empty(2, BATCH, dtype=torch.int32, device=device) for _ in range(2)]
    hl2 = [torch.zeros(1, dtype=torch.float32).pin_memory() for _ in range(2)]
    dl2 = [torch.zeros(1, device=device), torch.zeros(1, device=device)]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    seen = 0.0
    barrier()
    t0 = time.perf_counter()
    for i in range(step_calls):
        k = i & 1
        if i >= 2:
            done[k].synchronize()
            seen += float(hl2[k][0])
        dpairs2[k].copy_(hpairs[i % nb], non_blocking=True)
        s.step_sgns(dpairs2[k][0], dpairs2[k][1], dist, NEG, LR, dl2[k])
        hl2[k].copy_(dl2[k], non_blocking=True)
        done[k].record()
    for k in range(2):
        done[k].synchronize()
        seen += float(hl2[k][0])
    barrier()
    per_step_s = time.perf_counter() - t0
    e2e_steps_per_call = CHUNK
    if not e2e_steps:                                         # runs too short for one chunked call
        e2e_steps, e2e_s, e2e_steps_per_call = step_calls, per_step_s, 1

    # roofline of the dominant kernel (the fused step kernel) in the launch configuration that was timed above:
    # event pairs on its stream around every launch (one launch = the steps between two replica merges)
    hot_mask = torch.zeros(2 * VOCAB, dtype=torch.bool, device=device)
    if hot.numel():
        hot_mask[hot] = True
    cold_rows = []
    for i in range(0, nb, max(1, nb // 16)):              # data property: distinct non-replicated rows of a batch
        bc, bo = batch(i)
        s.step_sgns(bc, bo, dist, NEG, LR, loss)
        keys = torch.cat([bc.long(), bo.long(), s.last_negatives().long()])
        cold_rows.append(int((~hot_mask[torch.unique(keys)]).sum()))
    s.kernel_timing(True)
    run(0, args.steps)
    k_ms, k_launches = s.kernel_time()
    s.kernel_timing(False)
    steps_per_launch = args.steps / max(k_launches, 1)
    row_bytes = DIM * 4
    key_bytes = BATCH * 4 * (2 + NEG)
    alg_bytes = (key_bytes + 2 * row_bytes * float(np.mean(cold_rows))) * steps_per_launch
    logical_bytes = (key_bytes + 2 * row_bytes * BATCH * (NEG + 2)) * steps_per_launch
    update_bytes = row_bytes * BATCH * (NEG + 2) * steps_per_launch
    k_s = (k_ms / 1e3) / max(k_launches, 1)
    red_l2 = s.probe_reduction_rate(64 << 20, 20)          # update payload rate with L2-resident targets
    red_dram = s.probe_reduction_rate(2 << 30, 5)          # ... with targets streaming from DRAM
    traffic = NCU_TRAFFIC["bytes_per_launch"] if NCU_TRAFFIC["sgns_kernel_sha1"] == sgns_kernel_sha1() else None

    ms, e2e_s, per_step_s = max_over_ranks([ms, e2e_s, per_step_s], world, device)
    pairs = args.steps * BATCH * world
    value = aggregate_throughput(args.steps * BATCH * ACCESSES_PER_PAIR, ms / 1e3, world)
    out = {
        "metric": "key accesses/s (pull+push+sample)", "value": value, "unit": "key accesses/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_SGNS,
                   "workers": WORKERS, "l2": "tables (2.4 GB) larger than L2; no explicit flush",
                   "distinct_batches": nb, "replicas": world},
        "updates_per_s": pairs * UPDATES_PER_PAIR / (ms / 1e3),
        "pairs_per_s": pairs / (ms / 1e3),
        "final_loss": final_loss,
        "clocks": clk.summary(),
        "e2e": {"value": e2e_steps * BATCH * world * ACCESSES_PER_PAIR / e2e_s, "unit": "key accesses/s",
                "h2d_bytes_per_step": 2 * BATCH * 4, "d2h_bytes_per_step": 4, "steps": e2e_steps,
                "steps_per_call": e2e_steps_per_call,
                "one_call_per_step": {"value": step_calls * BATCH * world * ACCESSES_PER_PAIR / per_step_s,
                                      "unit": "key accesses/s", "steps": step_calls}},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "sgns_runs_kernel (fused step, 16 steps per launch)", "achieved": alg_bytes / k_s / 1e9,
                     "peak": hbm_peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": alg_bytes / k_s / 1e9 / hbm_peak, "traffic": traffic,
                     "algorithmic_bytes_per_launch": alg_bytes, "logical_bytes_per_launch": logical_bytes,
                     "logical_gbs": logical_bytes / k_s / 1e9, "kernel_us": k_s * 1e6,
                     "steps_per_launch": steps_per_launch,
                     "kernel_share_of_step": (k_ms / args.steps) / (ms / args.steps),
                     "distinct_cold_rows_per_batch": float(np.mean(cold_rows)),
                     "update_payload_gbs": update_bytes / k_s / 1e9,
                     "frac_of_l2_reduction_ceiling": update_bytes / k_s / 1e9 / red_l2,
                     "reduction_rate_l2_resident_gbs": red_l2, "reduction_rate_dram_gbs": red_dram},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = sgns_cpu_baseline(c, o, weights, hot, budget_s=12.0)
    return out


# --------------------------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm
# --------------------------------------------------------------------------------------------
def oracle_setup(weights, hot):
    import oracle
    o = oracle.Oracle(2 * VOCAB, DIM, workers=WORKERS, sync_interval=SYNC_EVERY)
    o.init_uniform(0, 1, 0.5 / DIM)
    o.set_management(inputs.u32(hot), oracle.REPLICATE)
    d = o.register_distribution(VOCAB, inputs.u32(weights), VOCAB, oracle.BOUNDED, U=U_REUSE, G=G_POOL, seed=7)
    return o, d


def sgns_cpu_baseline(c, o_keys, weights, hot, budget_s):
    orc, d = oracle_setup(weights, hot)
    hc, ho = inputs.u32(c), inputs.u32(o_keys)
    nb = len(hc) // BATCH
    t0 = time.perf_counter()
    done = 0
    while done < nb and time.perf_counter() - t0 < budget_s:
        j = done * BATCH
        orc.step_sgns(hc[j:j + BATCH], ho[j:j + BATCH], d, NEG, LR)
        done += 1
    dt = time.perf_counter() - t0
    return {"value": done * BATCH * ACCESSES_PER_PAIR / dt, "unit": "key accesses/s", "cores": 1, "kind": "oracle",
            "sample": f"first {done} batches of {BATCH} pairs of the same workload, full-size tables, "
                      f"{dt:.1f} s on one host thread (of {os.cpu_count()} cores)"}


def run_sgns_reference(args):
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    # bounded sample: the pairs of one step are a prefix of a batch, sized after a probe step so that the
    # whole run stays within a few minutes
    nb = min(args.steps + args.warmup, 512)
    c, o, counts, weights = make_sgns_data(dev, nb, seed=0)
    freq = torch.cat([counts, counts])
    hot = torch.argsort(freq, descending=True, stable=True)[: int(HOT_FRACTION * 2 * VOCAB)]
    orc, d = oracle_setup(weights.cpu(), hot.cpu())
    hc, ho = inputs.u32(c), inputs.u32(o)
    t0 = time.perf_counter()
    orc.step_sgns(hc[:BATCH], ho[:BATCH], d, NEG, LR)
    probe = time.perf_counter() - t0
    per_step = BATCH
    budget = 150.0
    if probe * (args.steps + args.warmup) > budget:
        per_step = max(64, int(BATCH * budget / (probe * (args.steps + args.warmup))) // 64 * 64)

    def step(i):
        j = (i % nb) * BATCH
        orc.step_sgns(hc[j:j + per_step], ho[j:j + per_step], d, NEG, LR)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    dt = time.perf_counter() - t0
    value = args.steps * per_step * ACCESSES_PER_PAIR / dt
    sample = (f"{per_step} pairs per step (of the workload's {BATCH}), full-size tables, single host thread "
              f"of {os.cpu_count()} cores")
    return {
        "impl": "reference", "metric": "key accesses/s (pull+push+sample)", "value": value, "unit": "key accesses/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_SGNS, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "key accesses/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "key accesses/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


# --------------------------------------------------------------------------------------------
# the parameter-server microbenchmark: 100M keys x 128 floats, batches of 1M keys ~ Zipf(s), top-k
# replicated, PullSample under the four schemes (stands in for the paper's Sections 5.5-5.7 sweeps)
# --------------------------------------------------------------------------------------------
def _time_calls(fn, reps, warm=3):
    """Mean device time of fn() in seconds: CUDA events on the current stream around `reps` calls."""
    for _ in range(warm):
        fn()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / 1e3 / reps


class PsSetup:
    """The store of the microbenchmark with its inputs: key batches per skew, update rows, output buffers, the four
    sampling distributions.  Keys of rank r (0-based, by true frequency) are `hot_keys[r]`; replicating the top k
    means the first k of them, in that order, so the most frequent key gets hot slot 0."""

    def __init__(self, binding, device, nk, seed=0, levels=PS_LEVELS):
        self.binding, self.device, self.nk, self.seed = binding, device, nk, seed
        self.N, self.L, self.row = PS_BATCH, PS_LEN, PS_LEN * 4
        self.s = binding.Store(nk, PS_LEN, workers=WORKERS, sync_interval=0, deterministic=False, track_ownership=True)
        self.s.init_uniform(0, 3, 0.1)
        self.hot_keys = inputs.rank_to_key(torch.arange(min(max(PS_TOPKS), nk), device=device), nk, seed=1).to(torch.int32).contiguous()
        self.topk = 0
        g = torch.Generator(device=device)
        g.manual_seed(17 + seed)
        self.delta = torch.randn(self.N, self.L, device=device, generator=g)
        self.out = torch.empty(self.N, self.L, device=device)
        self.skeys = torch.empty(self.N, dtype=torch.int32, device=device)
        self.svals = torch.empty(self.N, self.L, device=device)
        self._batches = {}
        self.dists = {}
        if levels:
            w = inputs.zipf_integer_weights(nk, 1.0, device).to(torch.int32).contiguous()
            lv = {"CONFORM": binding.CONFORM, "BOUNDED": binding.BOUNDED, "LONG-TERM": binding.LONGTERM,
                  "NON-CONFORM": binding.NONCONFORM}
            t0 = time.perf_counter()
            for name in levels:
                self.dists[name] = self.s.register_distribution(0, w, nk, lv[name], U=U_REUSE, G=G_POOL, seed=11 + lv[name])
            torch.cuda.synchronize()
            self.alias_build_s = (time.perf_counter() - t0) / len(levels)
            del w

    def batches(self, skew):
        """Four batches of 1M keys ~ Zipf(skew) over the store's keys (seeded; kept for the skew last asked for)."""
        if skew not in self._batches:
            self._batches.clear()
            cdf = inputs.zipf_cdf(self.nk, skew, self.device) if skew > 0 else None
            self._batches[skew] = [inputs.zipf_keys(self.N, self.nk, skew, 100 + 10 * self.seed + i, self.device, cdf=cdf)
                                   .to(torch.int32).contiguous() for i in range(4)]
            del cdf
        return self._batches[skew]

    def set_topk(self, k):
        k = min(k, self.hot_keys.numel())
        if k < self.topk:
            self.s.set_management(self.hot_keys[k:self.topk].contiguous(), self.binding.SINGLE)
        elif k > self.topk:
            self.s.set_management(self.hot_keys[self.topk:k].contiguous(), self.binding.REPLICATE)
        self.topk = k

    def distinct_cold(self, keys):
        """Distinct non-replicated keys of a batch: the rows that have to come from (and go back to) HBM."""
        u = torch.unique(keys.long())
        if self.topk:
            hot = torch.zeros(self.nk, dtype=torch.bool, device=self.device)
            hot[self.hot_keys[:self.topk].long()] = True
            u = u[~hot[u]]
            del hot
        return int(u.numel())

    def alg_bytes(self, kind, ucold):
        """Algorithmic bytes of one 1M-key launch: keys + the caller's rows + the distinct cold rows of the table
        (read once for a pull; read and written once for a push)."""
        N, row = self.N, self.row
        if kind == "pull":
            return 4 * N + row * N + row * ucold
        if kind == "push":
            return 4 * N + row * N + 2 * row * ucold
        if kind == "sample_rows":                    # keys read from the handle and written out, rows written, cold rows read
            return 8 * N + row * N + row * ucold
        raise ValueError(kind)

    def sample(self, level):
        h = self.s.prepare_sample(self.dists[level], self.N)
        self.s.pull_sample(h, self.N, True, self.skeys, self.svals)

    def close(self):
        self.s.close()
        for name in ("delta", "out", "svals", "skeys"):
            setattr(self, name, None)
        self._batches.clear()
        torch.cuda.empty_cache()


def ps_point(ps, skew, topk, reps, hbm_peak):
    """pull and push of 1M keys at one (skew, top-k) point: kernel time by event pairs on the launching stream."""
    s = ps.s
    batches = ps.batches(skew)
    ps.set_topk(topk)
    N, row = ps.N, ps.row
    ucold = float(np.mean([ps.distinct_cold(b) for b in batches]))
    s.kernel_timing(True)
    res = {}
    for op in ("pull", "push"):
        for i in range(3):
            (s.pull(batches[i % 4], ps.out) if op == "pull" else s.push(batches[i % 4], ps.delta))
        s.kernel_times()
        for i in range(reps):
            (s.pull(batches[i % 4], ps.out) if op == "pull" else s.push(batches[i % 4], ps.delta))
            if op == "push" and topk and (i + 1) % 16 == 0:
                s.sync()
        ms, n = s.kernel_times()[op]
        t = ms / 1e3 / n
        alg = ps.alg_bytes(op, ucold)
        res[op] = {"us": t * 1e6, "keys_per_s": N / t, "algorithmic_gbs": alg / t / 1e9, "frac": alg / t / 1e9 / hbm_peak,
                   "logical_gbs": (4 * N + (2 if op == "pull" else 3) * row * N) / t / 1e9}
    if topk:
        # pull again while the replicas hold unmerged updates (the pulls above saw freshly merged replicas)
        for i in range(4):
            s.push(batches[i % 4], ps.delta)
        s.kernel_times()
        for i in range(reps):
            s.pull(batches[i % 4], ps.out)
        ms, n = s.kernel_times()["pull"]
        t = ms / 1e3 / n
        alg = ps.alg_bytes("pull", ucold)
        res["pull_with_pending_updates"] = {"us": t * 1e6, "keys_per_s": N / t, "algorithmic_gbs": alg / t / 1e9,
                                            "frac": alg / t / 1e9 / hbm_peak}
        s.sync()
    s.kernel_timing(False)
    return {"zipf_s": skew, "topk": topk, "distinct_cold_rows": ucold, **res}


def ps_sync_point(ps, skew, topk, interval):
    """Pushes of 1M keys with a replica merge every `interval` pushes: device time per push, merges included."""
    s = ps.s
    batches = ps.batches(skew)
    ps.set_topk(topk)
    n_push = max(interval, 32)
    state = {"i": 0}

    def push_and_merge():
        for _ in range(n_push):
            s.push(batches[state["i"] % 4], ps.delta)
            state["i"] += 1
            if state["i"] % interval == 0:
                s.sync()
    t = _time_calls(push_and_merge, 2, warm=1) / n_push
    s.sync()
    return {"zipf_s": skew, "topk": topk, "merge_every": interval, "push_us_incl_merge": t * 1e6, "keys_per_s": ps.N / t}


def ps_sample_point(ps, level, reps, hbm_peak, warm=3):
    """PrepareSample + PullSample (keys and rows) of 1M keys from the Zipf(1.0) target under one scheme."""
    N, L = ps.N, ps.L
    t = _time_calls(lambda: ps.sample(level), max(reps, 1), warm=warm)
    uniq = int(torch.unique(ps.skeys).numel())
    draws = N // U_REUSE if level in ("BOUNDED", "LONG-TERM") else N        # pooled reuse draws every pool once
    alg = 4 * N + L * 4 * N + L * 4 * uniq + 16 * draws                     # keys out, rows out, distinct rows read, alias entries
    return {"level": level, "us": t * 1e6, "keys_per_s": N / t, "distinct_keys": uniq, "algorithmic_gbs": alg / t / 1e9,
            "frac": alg / t / 1e9 / hbm_peak}


def run_ps_sweep(args, device):
    """`--workload ps`: one JSON line per (skew, top-k) point."""
    from paper_2104_00501_b200 import binding
    hbm_peak, peak_kind = peaks()
    ps = PsSetup(binding, device, args.ps_keys, levels=())
    for skew in [float(x) for x in args.ps_skews.split(",")]:
        for topk in [int(x) for x in args.ps_topk.split(",")]:
            line = {"workload": "ps microbenchmark", "keys": ps.nk, "value_len": ps.L, "batch": ps.N, "peak": hbm_peak,
                    "peak_kind": peak_kind, **ps_point(ps, skew, topk, max(args.steps, 5), hbm_peak)}
            if topk:
                line["push_us_incl_merge_every"] = {str(iv): ps_sync_point(ps, skew, topk, iv)["push_us_incl_merge"]
                                                    for iv in PS_SYNCS}
            print(json.dumps(line), flush=True)
    ps.close()


def run_sample_sweep(args, device):
    """`--workload sample`: PullSample of 1M keys (keys + values) from a Zipf(1.0) target over the whole store."""
    from paper_2104_00501_b200 import binding
    hbm_peak, peak_kind = peaks()
    ps = PsSetup(binding, device, args.ps_keys)
    ps.set_topk(1000)
    for level in PS_LEVELS:
        print(json.dumps({"workload": "PullSample", "keys": ps.nk, "value_len": ps.L, "samples": ps.N, "peak_kind": peak_kind,
                          "alias_build_s": ps.alias_build_s,
                          **ps_sample_point(ps, level, args.steps, hbm_peak, warm=min(3, args.warmup))}), flush=True)
    ps.close()


def run_ps_line(args, rank, world, device):
    """The default line: pull + push + sample pull of 1M keys each per step on the 100M-key store."""
    from paper_2104_00501_b200 import binding
    hbm_peak, peak_kind = peaks()
    K, W = args.steps, args.warmup
    ps = PsSetup(binding, device, args.ps_keys, seed=rank)
    s, N, row = ps.s, ps.N, ps.row
    ps.set_topk(PS_TOPK)
    batches = ps.batches(PS_SKEW)
    state = {"pushes": 0}

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def step(i):
        s.pull(batches[i % 4], ps.out)
        s.push(batches[(i + 1) % 4], ps.delta)
        state["pushes"] += 1
        if state["pushes"] % PS_SYNC == 0:
            s.sync()
        ps.sample(PS_LEVEL)

    # warm-up (timed only to size the repetitions: the timed region repeats the K steps until it is a second long)
    step(0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(W):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    est_ms = e0.elapsed_time(e1) / W
    reps = int(min(max(5, -(-args.min_timed_ms // (est_ms * K))), max(5, 60000 // (4 * K))))
    reps = int(max_over_ranks([reps], world, device)[0])
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    launches0 = s.stats()["launches"]
    s.kernel_timing(True)
    s.kernel_times()                                            # start afresh
    s.kernel_timing(False)
    barrier()
    with ClockSampler(torch.cuda.current_device()) as clk:
        ev[0].record()
        for r in range(reps):
            # every fourth repetition carries the event pairs around its kernels that the roofline figures come from; the
            # others run as a caller's loop does (an event between two kernels keeps the second from becoming resident while
            # the first drains), and the median repetition, which `value` is taken from, is one of those
            timed_kernels = r % PS_KERNEL_EVENTS_EVERY == PS_KERNEL_EVENTS_EVERY - 1
            if timed_kernels:
                s.kernel_timing(True)
            for i in range(K):
                step(r * K + i)
            if timed_kernels:
                s.kernel_timing(False)
            ev[r + 1].record()
        barrier()
    rep_ms = [ev[r].elapsed_time(ev[r + 1]) for r in range(reps)]
    kt = s.kernel_times()
    launches = (s.stats()["launches"] - launches0) / reps
    assert s.status_check() == 0
    ms = float(np.median(rep_ms))                               # K steps
    total_ms = float(sum(rep_ms))

    # roofline of the three main kernels in the launch configuration that was just timed
    ucold = {"pull": float(np.mean([ps.distinct_cold(b) for b in batches]))}
    ucold["push"] = ucold["pull"]
    ucold["sample_rows"] = float(ps.distinct_cold(ps.skeys))
    kernels = {}
    for kind in ("pull", "push", "sample_rows"):
        k_ms, k_n = kt[kind]
        t = k_ms / 1e3 / max(k_n, 1)
        alg = ps.alg_bytes(kind, ucold[kind])
        name, m0, m1 = PS_KERNEL_SOURCE[kind]
        cap = NCU_TRAFFIC_PS[kind]
        traffic = (cap["dram_bytes"] * alg / cap["algorithmic_bytes"] if cap["sha1"] == kernel_source_sha1(m0, m1) else None)
        kernels[kind] = {"kernel": name, "kernel_us": t * 1e6, "launches": int(k_n), "achieved": alg / t / 1e9,
                         "frac": alg / t / 1e9 / hbm_peak, "algorithmic_bytes_per_launch": alg,
                         "distinct_cold_rows": ucold[kind], "traffic": traffic,
                         "share_of_step": (k_ms / max(k_n, 1)) / (ms / K)}
    draw_ms, draw_n = kt["draw"]
    dominant = max(kernels, key=lambda k: kernels[k]["kernel_us"])
    dk = kernels[dominant]

    # end to end through the public API with HOST buffers: every step's keys and update rows start in pinned host memory
    # and are copied to the device inside the timed region, and every step's results (pulled rows, sampled keys and
    # rows) are copied back to pinned host memory, where the host looks at them.  Two sets of buffers and three streams
    # (copies in, the library's calls, copies out), so that a step's copies overlap its neighbours' work as a real caller
    # would arrange it; every byte still crosses the link inside the timed region.
    e2e_steps = max(4, min(K, 32))
    hk = [b.cpu().pin_memory() for b in batches]
    hdelta = ps.delta.cpu().pin_memory()
    hout = [torch.empty((N, ps.L), dtype=torch.float32).pin_memory() for _ in range(2)]
    hsvals = [torch.empty((N, ps.L), dtype=torch.float32).pin_memory() for _ in range(2)]
    hskeys = [torch.empty(N, dtype=torch.int32).pin_memory() for _ in range(2)]
    dk_pull = [torch.empty_like(batches[0]) for _ in range(2)]
    dk_push = [torch.empty_like(batches[0]) for _ in range(2)]
    ddelta = [torch.empty_like(ps.delta) for _ in range(2)]
    dout = [ps.out, torch.empty_like(ps.out)]
    dskeys = [ps.skeys, torch.empty_like(ps.skeys)]
    dsvals = [ps.svals, torch.empty_like(ps.svals)]
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    dist_id = ps.dists[PS_LEVEL]

    def e2e_loop(steps, rows_cross):
        h2d = [torch.cuda.Event() for _ in range(2)]
        done = [torch.cuda.Event() for _ in range(2)]
        d2h = [torch.cuda.Event() for _ in range(2)]
        seen = 0.0
        barrier()
        t0 = time.perf_counter()
        for i in range(steps):
            k = i & 1
            if i >= 2:                                         # the results of step i - 2 have landed: the host reads them
                d2h[k].synchronize()
                seen += float(hskeys[k][0]) + (float(hout[k][0, 0]) + float(hsvals[k][-1, -1]) if rows_cross else 0.0)
                s_in.wait_event(done[k])                       # ... and that step's inputs may be overwritten
            with torch.cuda.stream(s_in):
                dk_pull[k].copy_(hk[i % 4], non_blocking=True)
                dk_push[k].copy_(hk[(i + 1) % 4], non_blocking=True)
                if rows_cross:
                    ddelta[k].copy_(hdelta, non_blocking=True)
                h2d[k].record(s_in)
            main.wait_event(h2d[k])
            if i >= 2:
                main.wait_event(d2h[k])                        # the output buffers of step i - 2 have been copied out
            s.pull(dk_pull[k], dout[k])
            s.push(dk_push[k], ddelta[k] if rows_cross else ps.delta)
            state["pushes"] += 1
            if state["pushes"] % PS_SYNC == 0:
                s.sync()
            s.pull_sample(s.prepare_sample(dist_id, N), N, True, dskeys[k], dsvals[k])
            done[k].record(main)
            s_out.wait_event(done[k])
            with torch.cuda.stream(s_out):
                hskeys[k].copy_(dskeys[k], non_blocking=True)
                if rows_cross:
                    hout[k].copy_(dout[k], non_blocking=True)
                    hsvals[k].copy_(dsvals[k], non_blocking=True)
                d2h[k].record(s_out)
        for k in range(2):
            d2h[k].synchronize()
            seen += float(hskeys[k][0]) + (float(hout[k][0, 0]) + float(hsvals[k][-1, -1]) if rows_cross else 0.0)
        barrier()
        dt = time.perf_counter() - t0
        assert np.isfinite(seen)
        return dt

    e2e_loop(2, True)
    e2e_s = e2e_loop(e2e_steps, True)
    keys_steps = max(e2e_steps, min(4 * K, 256))
    keys_s = e2e_loop(keys_steps, False)       # only keys cross the bus: update rows and results stay on the device

    ms, total_ms, e2e_s, keys_s = max_over_ranks([ms, total_ms, e2e_s, keys_s], world, device)
    acc_step = 3 * N                                            # pulled + pushed + sampled keys
    out = {
        "metric": "key accesses/s (pull+push+sample)", "value": aggregate_throughput(K * acc_step, ms / 1e3, world),
        "unit": "key accesses/s", "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms / K,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_PS, "workers": WORKERS, "keys": ps.nk, "value_len": ps.L, "batch": N,
                   "l2": "inputs (three 512 MB row buffers, 51 GB table) larger than L2; no explicit flush",
                   "timed_region": f"median of {reps} back-to-back repetitions of the {K} steps ({total_ms:.0f} ms in all); every "
                                   f"{PS_KERNEL_EVENTS_EVERY}th repetition has event pairs around its kernels (the roofline figures)",
                   "replicas": world},
        "updates_per_s": aggregate_throughput(K * N, ms / 1e3, world),
        "repetitions": reps, "timed_ms_total": total_ms,
        "clocks": clk.summary(),
        "e2e": {"value": aggregate_throughput(e2e_steps * acc_step, e2e_s, world), "unit": "key accesses/s",
                "h2d_bytes_per_step": 4 * N + 4 * N + row * N, "d2h_bytes_per_step": row * N + 4 * N + row * N,
                "steps": e2e_steps,
                "note": "keys, update rows, pulled rows, sampled keys and rows all cross the bus (copies in, calls and copies out on three streams, two buffer sets): bound by the host link",
                "keys_only": {"value": aggregate_throughput(keys_steps * acc_step, keys_s, world), "unit": "key accesses/s",
                              "h2d_bytes_per_step": 8 * N, "d2h_bytes_per_step": 4 * N, "steps": keys_steps,
                              "note": "update rows and pulled/sampled rows stay on the device (a trainer on the GPU)"}},
        "gpu_launches": int(round(launches)),
        "roofline": {"bound": "hbm", "kernel": f"{dk['kernel']} ({dominant})", "achieved": dk["achieved"], "peak": hbm_peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": dk["frac"], "traffic": dk["traffic"],
                     "traffic_note": "ncu DRAM bytes of a 1M-key launch on a 4M-key table, scaled by the algorithmic bytes",
                     "algorithmic_bytes_per_launch": dk["algorithmic_bytes_per_launch"], "kernel_us": dk["kernel_us"],
                     "kernels": kernels, "draw_kernel_us": draw_ms / max(draw_n, 1) * 1e3},
    }
    if rank == 0 and world == 1 and not args.no_sweep:
        out["sweep"] = ps_sweep(args, ps, hbm_peak, device)
    ps.close()
    if rank == 0 and world == 1 and not args.no_sweep:
        out["sweep"]["steps"] = step_entries(args, device)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = ps_cpu_baseline(budget_s=12.0)
    return out


def ps_sweep(args, ps, hbm_peak, device):
    """Every grid point of the microbenchmark: 4 skews x 3 top-k (pull and push), 3 merge intervals, 4 sampling
    schemes.  Kernel times by event pairs; fractions are algorithmic bytes over the measured copy peak."""
    reps = max(min(args.steps, 20), 10)
    sampling = [ps_sample_point(ps, level, reps, hbm_peak) for level in PS_LEVELS]          # at the headline's top-1k
    merges = [ps_sync_point(ps, PS_SKEW, PS_TOPK, iv) for iv in PS_SYNCS]
    points = [ps_point(ps, skew, topk, reps, hbm_peak) for skew in PS_SKEWS for topk in PS_TOPKS]
    return {"pull_push": points, "merge_interval": merges, "pull_sample": sampling, "alias_build_s": ps.alias_build_s,
            "reps_per_point": reps}


def step_entries(args, device):
    """One entry per workload step (skip-gram, ComplEx, matrix factorization) at the paper-sized configurations."""
    out = {}
    try:
        out["sgns"] = sgns_entry(device, steps=256)
        out["complex"] = run_step_workload(args, device, "kge", emit=False)
        out["mf"] = run_step_workload(args, device, "mf", emit=False)
        mo, args.mf_order = args.mf_order, "column"
        out["mf_by_column"] = run_step_workload(args, device, "mf", emit=False)
        args.mf_order = mo
    finally:
        torch.cuda.empty_cache()
    return out


def sgns_entry(device, steps):
    """The skip-gram workload in brief: `steps` steps through nups_run_sgns, 64 per call."""
    from paper_2104_00501_b200 import binding
    nb = steps
    s, dist, hot, c, o, weights = build_store(binding, device, nb, seed=0)
    losses = torch.zeros(64, dtype=torch.float32, device=device)

    def run():
        for j in range(0, nb, 64):
            s.run_sgns(c[j * BATCH:(j + 64) * BATCH], o[j * BATCH:(j + 64) * BATCH], BATCH, dist, NEG, LR, losses)
    dt = _time_calls(run, 3, warm=1) / nb
    s.kernel_timing(True)
    run()
    k_ms, k_n = s.kernel_times()["step"]
    s.kernel_timing(False)
    s.close()
    return {"workload": WORKLOAD_SGNS, "us_per_step": dt * 1e6, "key_accesses_per_s": BATCH * ACCESSES_PER_PAIR / dt,
            "updates_per_s": BATCH * UPDATES_PER_PAIR / dt, "kernel": "sgns_runs_kernel", "kernel_us_per_launch": k_ms / max(k_n, 1) * 1e3,
            "steps_per_launch": nb / max(k_n, 1), "final_loss": float(losses.mean())}


# --------------------------------------------------------------------------------------------
# the oracle on the microbenchmark: CPU baseline and reference arm
# --------------------------------------------------------------------------------------------
class PsOracle:
    """The oracle on the same kind of step, with the table scaled down to PS_ORACLE_KEYS keys (a 51 GB table on the
    host is not something every box has): keys ~ Zipf(1.0) over the smaller key space, the same top-1k replicated."""

    def __init__(self, n_max):
        import oracle
        nk = PS_ORACLE_KEYS
        self.o = oracle.Oracle(nk, PS_LEN, workers=WORKERS)
        self.o.init_uniform(0, 3, 0.1)
        hot = inputs.u32(inputs.rank_to_key(torch.arange(PS_TOPK), nk, seed=1))
        self.o.set_management(hot, oracle.REPLICATE)
        w = inputs.u32(inputs.zipf_integer_weights(nk, 1.0, "cpu"))
        self.d = self.o.register_distribution(0, w, nk, oracle.BOUNDED, U=U_REUSE, G=G_POOL, seed=13)
        cdf = inputs.zipf_cdf(nk, PS_SKEW, "cpu")
        self.keys = [inputs.u32(inputs.zipf_keys(n_max, nk, PS_SKEW, 100 + i, "cpu", cdf=cdf)) for i in range(2)]
        self.delta = np.random.default_rng(0).standard_normal((n_max, PS_LEN), dtype=np.float32)
        self.pushes = 0

    def step(self, i, n):
        self.o.pull(self.keys[i % 2][:n])
        self.o.push(self.keys[(i + 1) % 2][:n], self.delta[:n])
        self.pushes += 1
        if self.pushes % PS_SYNC == 0:
            self.o.sync()
        self.o.pull_sample(self.o.prepare_sample(self.d, n), n, values=True)

    @staticmethod
    def scaling():
        return (f"table scaled to {PS_ORACLE_KEYS:,} keys x {PS_LEN} fp32 (2 GB of host memory instead of 51 GB), keys ~ Zipf(1.0) "
                f"over them, top-1k replicated, same step otherwise")


def ps_cpu_baseline(budget_s):
    n = 65536
    orc = PsOracle(n)
    orc.step(0, 4096)
    t0 = time.perf_counter()
    done = 0
    while time.perf_counter() - t0 < budget_s:
        orc.step(done, n)
        done += 1
    dt = time.perf_counter() - t0
    return {"value": done * 3 * n / dt, "unit": "key accesses/s", "cores": 1, "kind": "oracle",
            "sample": f"{done} steps of {n} keys per pull, push and sample pull (the workload's steps take {PS_BATCH}), "
                      f"{PsOracle.scaling()}; {dt:.1f} s on one host thread (of {os.cpu_count()} cores)"}


def run_ps_reference(args):
    """`--impl reference`: the oracle, as it stands, on the default line's workload; every step a bounded sample."""
    total = args.steps + args.warmup
    orc = PsOracle(PS_BATCH)
    probe_n = 16384
    t0 = time.perf_counter()
    orc.step(0, probe_n)
    probe = time.perf_counter() - t0
    budget = 150.0
    per_step = int(min(PS_BATCH, max(4096, probe_n * budget / (probe * total) // 4096 * 4096)))
    for i in range(args.warmup):
        orc.step(i, per_step)
    t0 = time.perf_counter()
    for i in range(args.steps):
        orc.step(args.warmup + i, per_step)
    dt = time.perf_counter() - t0
    value = args.steps * 3 * per_step / dt
    sample = (f"{per_step} keys per pull, push and sample pull per step (of the workload's {PS_BATCH}), {PsOracle.scaling()}; "
              f"single host thread of {os.cpu_count()} cores")
    return {
        "impl": "reference", "metric": "key accesses/s (pull+push+sample)", "value": value, "unit": "key accesses/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_PS, "workers": WORKERS, "keys": PS_KEYS, "value_len": PS_LEN, "batch": PS_BATCH,
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": "key accesses/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "key accesses/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def run_shard_sweep(args, device):
    """The partitioned table on ONE GPU: 8 shards (every shard its own allocation, wired by address) standing in for 8
    ranks, 1M-key Zipf batches pulled and pushed through one rank's table.  All shards are local HBM here, so this
    measures the kernels' addressing, not NVLink: on several GPUs (N - 1) / N of the rows cross the links."""
    from paper_2104_00501_b200 import binding, sharded
    hbm_peak, peak_kind = peaks()
    nk, n_shards, L, N = args.ps_keys, 8, PS_LEN, PS_BATCH
    tables = [binding.ShardTable(nk, L, n_shards, j) for j in range(n_shards)]
    sharded.connect_local(tables)
    t = tables[0]
    g = torch.Generator(device=device)
    g.manual_seed(17)
    delta = torch.randn(N, L, device=device, generator=g)
    out = torch.empty(N, L, device=device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for skew in [float(x) for x in args.ps_skews.split(",")]:
        cdf = inputs.zipf_cdf(nk, skew, device) if skew > 0 else None
        batches = [inputs.zipf_keys(N, nk, skew, 100 + i, device, cdf=cdf).to(torch.int32).contiguous() for i in range(4)]
        del cdf
        ucold = float(np.mean([torch.unique(b.long()).numel() for b in batches]))
        line = {"workload": "partitioned table, 8 shards on one GPU: %d keys x %d fp32, 1M-key batches ~ Zipf(%.1f)" % (nk, L, skew),
                "zipf_s": skew, "distinct_rows": ucold, "peak_kind": peak_kind}
        for kind, call in (("pull", lambda b: t.pull(b, out)), ("push", lambda b: t.push(b, delta))):
            for b in batches:
                call(b)
            torch.cuda.synchronize()
            reps = 20
            e0.record()
            for r in range(reps):
                call(batches[r % 4])
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / reps
            alg = 4 * N + L * 4 * N + (1 if kind == "pull" else 2) * L * 4 * ucold
            line[kind] = {"us": us, "keys_per_s": N / us * 1e6, "algorithmic_gbs": alg / us / 1e3, "frac": alg / us / 1e3 / hbm_peak}
        assert t.status_check() == 0
        print(json.dumps(line), flush=True)
    for x in tables:
        x.close()


def run_staleness_sweep(args, device):
    """The SGNS workload with replicas merged by step count (every 16 batches) or by time: throughput and loss after
    the same number of steps from the same start values.  The periods span the paper's staleness experiment (125, 25
    and 5 merges per second, never) and, because a step takes about 10 us here, much shorter ones: what matters for
    the model is how many updates a replica absorbs between two merges."""
    from paper_2104_00501_b200 import binding
    steps = max(args.steps, 32768)
    nb = MAX_DISTINCT_BATCHES
    CHUNK = 64
    losses = torch.zeros(CHUNK, dtype=torch.float32, device=device)
    settings = [("every 16 steps", SYNC_EVERY, 0)] + [(f"every {us / 1000:g} ms", 0, us)
                                                      for us in (150, 500, 2_000, 8_000, 40_000, 200_000)] + [("never", 0, 0)]
    store, prev_interval = None, None
    for name, interval, period_us in settings:
        if store is None or interval != prev_interval:
            if store is not None:
                store.close()
            store, dist, hot, c, o, weights = build_store(binding, device, nb, seed=0, sync_interval=interval,
                                                          clip_factor=args.clip_factor)
            prev_interval = interval
        else:
            store.sync()
            store.init_uniform(0, 1, 0.5 / DIM)
        store.set_sync_period(period_us)

        def run(count):
            done = 0
            while done < count:
                j = done % nb
                m = min(CHUNK, count - done, nb - j)
                store.run_sgns(c[j * BATCH:(j + m) * BATCH], o[j * BATCH:(j + m) * BATCH], BATCH, dist, NEG, LR, losses[:m])
                done += m
        run(args.warmup)
        m0 = store.stats()["background_merges"]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        run(steps)
        e1.record()
        torch.cuda.synchronize()
        t = e0.elapsed_time(e1) / 1e3
        st = store.stats()
        store.set_sync_period(0)
        print(json.dumps({"workload": "SGNS, replica staleness", "merge": name, "clip_factor": args.clip_factor,
                          "steps": steps, "seconds": t,
                          "key_accesses_per_s": steps * BATCH * ACCESSES_PER_PAIR / t, "us_per_step": t / steps * 1e6,
                          "background_merges": st["background_merges"] - m0, "loss_last_64_steps": float(losses.mean())}),
              flush=True)
    store.close()


def run_step_workload(args, device, which, emit=True):
    """ComplEx + AdaGrad (config 3) or matrix factorization (config 4) steps in fast mode."""
    from paper_2104_00501_b200 import binding
    hbm_peak, peak_kind = peaks()
    loss = torch.zeros(1, device=device)
    reps = max(args.steps, 20)
    if which == "kge":
        E, Rl, L, B, K = args.kge_entities, 1000, 500, 8192, 10
        s = binding.Store(E + Rl, L, workers=WORKERS, sync_interval=SYNC_EVERY, deterministic=False, with_adagrad=True)
        s.init_uniform(0, 5, 0.05)
        nb = 64
        h, r, t = inputs.kge_triples(nb * B, E, Rl, 0.9, 1.2, 0, device)
        h, r, t = (x.to(torch.int32).contiguous() for x in (h, r, t))
        s.count_accesses(torch.cat([h, t]))
        hot = s.select_hot(False, 100)                               # the 100 x mean rule on the entities ...
        rel = torch.arange(E, E + Rl, device=device, dtype=torch.int32)
        s.set_management(torch.cat([rel, hot]).contiguous(), binding.REPLICATE)   # ... and every relation
        dist = s.register_distribution(0, None, E, binding.CONFORM, seed=3)
        state = {"i": 0}

        def step():
            j = (state["i"] % nb) * B
            state["i"] += 1
            s.step_complex(h[j:j + B], r[j:j + B], t[j:j + B], dist, K, 0.1, 1e-10, loss)
        per_item, upd, rows_per_item = 3 + K + (K + 3), K + 3, 2 * (K + 3)
        name, cfg = "complex_kernel", f"ComplEx+AdaGrad: 5M entities, 1000 relations, 500 fp32/row + accumulator, batch {B}, {K} negatives"
    else:
        M, N, L, B = args.mf_rows, args.mf_rows // 10, 100, 65536
        s = binding.Store(M + N, L, workers=WORKERS, sync_interval=SYNC_EVERY, deterministic=False)
        s.init_uniform(0, 5, 0.3)
        nb = 32
        i, j, x = inputs.mf_cells(nb * B, M, N, 0.8, 100, 0.1, 0, device)
        i, j, x = i.to(torch.int32).contiguous(), j.to(torch.int32).contiguous(), x.contiguous()
        s.count_accesses(torch.cat([i, j]))                         # the hot set comes from independent draws ...
        hot = s.select_hot(False, 100)
        if hot.numel():
            s.set_management(hot, binding.REPLICATE)
        if args.mf_order != "random":                                # ... the steps may visit the cells column by column
            i, j, x = inputs.mf_cells(nb * B, M, N, 0.8, 100, 0.1, 0, device, by_column_of=100 * M)
            i, j, x = i.to(torch.int32).contiguous(), j.to(torch.int32).contiguous(), x.contiguous()
        state = {"i": 0}

        def step():
            a = (state["i"] % nb) * B
            state["i"] += 1
            s.step_mf(i[a:a + B], j[a:a + B], x[a:a + B], 1e-4, 0.01, loss, by_column=args.mf_order == "column")     # "column-plain": the same cells through nups_step_mf
        per_item, upd, rows_per_item = 4, 2, 2
        name, cfg = ("mf_runs_kernel" if args.mf_order == "column" else "mf_kernel"), f"MF: 10M x 1M, rank 100, batch {B}, L2 0.01, cells in {args.mf_order} order"
    dt = _time_calls(step, reps)
    s.kernel_timing(True)
    _time_calls(step, reps, warm=0)
    k_ms, k_n = s.kernel_time()
    s.kernel_timing(False)
    k_s = k_ms / 1e3 / max(k_n, 1)
    tables = 2 if which == "kge" else 1
    logical = B * rows_per_item * L * 4 * 2 * (1 if which == "mf" else 1)      # every touched row read and written once
    # What the atomic update path allows: nearly all rows of these steps are cold, so every row is read once (at best
    # at the copy peak) and every update is a floating-point reduction to a DRAM-resident row, whose rate the library
    # measures by itself.  floor = both in full overlap, read_then_reduce = one after the other.
    red_dram = s.probe_reduction_rate(2 << 30, 5)
    t_read, t_red = (logical / 2) / (hbm_peak * 1e9), (logical / 2) / (red_dram * 1e9)
    line = {"workload": cfg, "kernel": name, "hot_slots": s.stats()["hot_slots"], "us_per_step": dt * 1e6,
            "kernel_us": k_s * 1e6, "key_accesses_per_s": B * per_item / dt, "updates_per_s": B * upd / dt,
            "logical_gbs": logical / k_s / 1e9, "logical_frac_of_hbm_peak": logical / k_s / 1e9 / hbm_peak,
            "reduction_rate_dram_gbs": red_dram, "floor_us_reads_and_reductions_overlapped": max(t_read, t_red) * 1e6,
            "us_read_then_reduce": (t_read + t_red) * 1e6,
            "frac_of_overlapped_floor": max(t_read, t_red) / k_s,
            "peak_kind": peak_kind, "final_loss": float(loss.item()), "tables": tables}
    s.close()
    if emit:
        print(json.dumps(line), flush=True)
    return line


def main():
    global TOKENS, HOT_FRACTION, WORKERS
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="default line only: skip the sweep of the other grid points")
    ap.add_argument("--min-timed-ms", type=float, default=1250.0,
                    help="the timed region repeats the K steps until it is at least this long (at least 5 times)")
    ap.add_argument("--workload", default="psline", choices=["psline", "sgns", "ps", "sample", "kge", "mf", "staleness", "shard"],
                    help="psline (default): the parameter-server microbenchmark line with its sweep; sgns: the skip-gram line; "
                         "the others print their own lines")
    ap.add_argument("--hot-fraction", type=float, default=HOT_FRACTION, help="share of keys to replicate (default 0.01)")
    ap.add_argument("--workers", type=int, default=WORKERS)
    ap.add_argument("--clip-factor", type=float, default=0.0,
                    help="staleness workload: clip replicated-key updates at this multiple of their mean norm")
    ap.add_argument("--tokens", type=int, default=TOKENS, help="length of the synthetic token stream (profiling runs use less)")
    ap.add_argument("--ps-keys", type=int, default=PS_KEYS, help="smaller for profiling runs")
    ap.add_argument("--kge-entities", type=int, default=5_000_000, help="smaller for profiling runs")
    ap.add_argument("--mf-rows", type=int, default=10_000_000, help="smaller for profiling runs")
    ap.add_argument("--mf-order", default="random", choices=["random", "column", "column-plain"],
                    help="mf: independent cells, or the first cells of a 1G-cell data set visited column by column "
                         "(column-plain: those cells through the step call for independent cells)")
    ap.add_argument("--ps-skews", default="0,0.6,1.0,1.4")
    ap.add_argument("--ps-topk", default="0,1000,100000")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    TOKENS = max(args.tokens, 10_000_000)
    HOT_FRACTION, WORKERS = args.hot_fraction, args.workers
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            line = run_sgns_reference(args) if args.workload == "sgns" else run_ps_reference(args)
            print(json.dumps(line), flush=True)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if args.workload == "ps":
        run_ps_sweep(args, device)
        return
    if args.workload == "sample":
        run_sample_sweep(args, device)
        return
    if args.workload in ("kge", "mf"):
        run_step_workload(args, device, args.workload)
        return
    if args.workload == "staleness":
        run_staleness_sweep(args, device)
        return
    if args.workload == "shard":
        run_shard_sweep(args, device)
        return
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=device)
    out = run_sgns_line(args, rank, world, device) if args.workload == "sgns" else run_ps_line(args, rank, world, device)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
