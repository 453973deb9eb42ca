#!/usr/bin/env python
"""Benchmark of the DES sparse step (find-or-insert, per-shard partials, shard
reduction + F, backward scatter + optimizer) on synthetic CTR-shaped batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl reference]

One JSON line on stdout (rank 0).  `value` = samples/s of the whole job with
the batch already resident in HBM; `e2e` = the same step from pinned host
buffers through des_step_host_submit / des_step_host_wait (H2D of the batch and
D2H of the aggregated outputs inside the timed region, every step; the copy of
one step overlaps the kernels of the step before; the blocking des_step_host
is timed beside it); `roofline` = the kernel with the largest share of the
step against the measured HBM copy bandwidth; `cpu_baseline` = the CPU oracle,
as it stands, on a bounded sample of the same batch.

With N > 1 (launched by torch.distributed.run) every rank runs its own replica
of the table on its own batches — the path has no exchange between GPUs — and
the job's samples/s is N * B over the slowest rank's time ("weak" scaling)."""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1909_04823_b200 import synth  # noqa: E402
from paper_1909_04823_b200.synth import OP_DENSE1, OP_FM, OP_LR, OP_POOL, PART_FIELD  # noqa: E402

METRIC = "samples/sec per DES fwd+bwd sparse step"
UNIT = "samples/s"


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, "measured" | "fallback")"""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", 1400.0)), "measured"
        except Exception:
            pass
    return 6650.0, 1400.0, "fallback"


def rows_per_shard(w, cap_total):
    if w.partition != PART_FIELD:
        return None
    cat = max(1, w.fields - w.bucket_fields)
    out = [256] * w.shards
    for f in range(w.fields):
        n = 64 if f < w.bucket_fields else cap_total // cat
        out[f % w.shards] += int(n * 1.05) + 64
    return out


def per_rank_workload(w, rank, world):
    """Replicas are independent: rank r draws its own batches (seed offset), same shapes."""
    return w if world == 1 else w.scaled(seed=w.seed + 1000 * rank)


def max_over_ranks(value, world, device=None):
    """Slowest rank's time (the job's step time) — torch.distributed MAX all-reduce."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(batch, world, ms_step):
    return world * batch / (ms_step / 1e3)


def sub_batch(b, n_samples):
    """The first n_samples samples of a batch (a bounded sample for the CPU leg)."""
    F = b.fields
    end = int(b.offsets[n_samples * F])
    return synth.Batch(n_samples, F, b.offsets[:n_samples * F + 1].copy(), b.ids[:end].copy(),
                       None if b.vals is None else b.vals[:end].copy())


# ---------------------------------------------------------------------------
def oracle_step(o, w, b, g):
    fi = o.find_or_insert(b)
    part = o.forward_partials(w.ops, b, fi, want_pooled=bool(w.ops & (OP_POOL | OP_DENSE1)),
                              want_dense=bool(w.ops & OP_DENSE1))
    agg = o.aggregate(b.batch, part)
    pooled = None if agg["pooled"] is None else agg["pooled"].astype(np.float32)
    o.backward_update(w.ops, b, fi, agg["A"].astype(np.float32), pooled, g.get("gL"), g.get("gF"),
                      g.get("gE") if (w.ops & OP_POOL) else None, g.get("gZ") if (w.ops & OP_DENSE1) else None)


def time_oracle(w, batch, grads, budget_s=15.0, steps=1, warmup=0, omp=False):
    """Times the CPU oracle on the first Bs samples of `batch`, Bs sized so that
    one step takes about budget_s seconds.  omp: the same source compiled with
    -fopenmp, on all host cores.  Returns (samples/s, Bs, seconds per step)."""
    from oracle import Oracle
    if w.hidden:
        W1 = synth.dense1_weights(w)

    def run(bs, n):
        sb = sub_batch(batch, bs)
        g = {k_: v[:bs] for k_, v in grads.items()}
        o = Oracle.for_workload(w, omp=omp)
        if w.hidden:
            o.dense1_set(W1)
        ts = []
        for _ in range(n):
            t0 = time.perf_counter()
            oracle_step(o, w, sb, g)
            ts.append(time.perf_counter() - t0)
        o.close()
        return ts

    probe = max(1, min(batch.batch, 64 if omp else 8))
    t = run(probe, 1)[0]
    per_sample = max(t / probe, 1e-7)
    bs = int(max(1, min(batch.batch, budget_s / per_sample)))
    ts = run(bs, warmup + steps)[warmup:]
    sec = float(np.mean(ts))
    return bs / sec, bs, sec


# ---------------------------------------------------------------------------
class ClockSampler:
    """SM clock, power and throttle reasons of one GPU, sampled every 20 ms by a thread (NVML, read-only
    queries) with host time stamps, so that every timed window gets its own median clock."""
    REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"), (0x4, "sw_power_cap"))

    def __init__(self, torch_index):
        import threading
        self.samples = []           # (time, sm MHz, reasons bitmask, watts)
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            h = None
            try:
                uuid = str(torch.cuda.get_device_properties(torch_index).uuid)
                h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByIndex(torch_index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(pynvml, "nvmlDeviceGetCurrentClocksThrottleReasons")

            def loop():
                while not self._stop.is_set():
                    try:
                        self.samples.append((time.perf_counter(), float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)),
                                             int(reasons_fn(h)), pynvml.nvmlDeviceGetPowerUsage(h) / 1e3))
                    except Exception:
                        pass
                    self._stop.wait(0.02)
            self._thread = threading.Thread(target=loop, daemon=True)
            self._thread.start()
        except Exception as ex:
            log(f"[bench] clock sampling unavailable: {ex!r}")

    def window(self, t0, t1):
        """Median SM MHz and the throttle reasons seen between two host time stamps."""
        sel = [s for s in self.samples if t0 <= s[0] <= t1]
        if not sel:   # a window shorter than the sampling period: the nearest sample
            sel = sorted(self.samples, key=lambda s_: abs(s_[0] - 0.5 * (t0 + t1)))[:1]
        if not sel:
            return {"sm_mhz": None, "reasons": [], "samples": 0}
        bits = 0
        for s_ in sel:
            bits |= s_[2]
        return {"sm_mhz": float(np.median([s_[1] for s_ in sel])), "samples": len(sel),
                "reasons": sorted(n for b, n in self.REASONS if bits & b)}

    def stop(self, windows=None):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": []}
        sel = self.samples
        if windows:
            inw = [s_ for s_ in self.samples if any(a <= s_[0] <= b for a, b in windows)]
            sel = inw or sel
        bits = 0
        for s_ in sel:
            bits |= s_[2]
        return {"sm_mhz": float(np.median([s_[1] for s_ in sel])), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(n for b, n in self.REASONS if bits & b), "samples": len(sel),
                "power_w_max": round(max(s_[3] for s_ in sel), 1), "scope": "timed windows only" if windows else "whole run"}


# ---------------------------------------------------------------------------
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from an ncu capture of the benchmark's
# own batch on a 4e6-key table (the 2e8-key table cannot be captured under multi-pass replay).  The scatter's traffic does not depend on
# the table; kernels that touch table rows move fewer DRAM bytes there (U = 1.06 M instead of 1.81 M).
NCU_DRAM_TRAFFIC = {
    ("cfg5", "grad_scatter_kernel"): 1807e6,
    ("cfg5", "super_dense_kernel"): 533e6,
    ("cfg5", "shard_partials_kernel"): 962e6,
    ("cfg5", "pool_kernel"): 1213e6,
    ("cfg5", "update_rows_kernel"): 1933e6,
    ("cfg5", "probe_claim_kernel"): 596e6,
    ("cfg5", "flag_count_kernel"): 566e6,
    ("cfg5", "resolve_kernel"): 421e6,
    ("cfg5", "make_dest_kernel"): 225e6,
    ("cfg5", "route_kernel"): 456e6,
    ("cfg5", "single_gather_kernel"): 1290e6,
    ("cfg5", "fused_finish_kernel"): 440e6,
}


def kernel_bytes(name, st):
    """Algorithmic bytes one launch of `name` must move (what the method needs,
    each datum once: ids, offsets and index arrays per occurrence, table rows per unique key)."""
    nnz, B, F, k, S, U, R = st["nnz"], st["B"], st["F"], st["k"], st["S"], st["U"], st["rep_rows"]
    row = 4 * k + 16
    state = 1 if st["adagrad"] else 0
    small = bool(st["ops"] & (OP_LR | OP_FM))
    pool = bool(st["ops"] & (OP_POOL | OP_DENSE1))
    if name == "probe_claim_kernel":
        return 8 * nnz + 16 * U + 4 * nnz + nnz
    if name == "flag_count_kernel":      # slot index and shard in; the slot's (row, scratch); flag, row, first occurrence out
        return 4 * nnz + nnz + 8 * U + nnz + 4 * nnz + 4 * nnz
    if name == "assign_kernel":          # exits at once when the batch has no new key (a populated table)
        return (nnz + nnz + 4 * U + 8 * U + 4 * U) if st.get("new_keys", True) else None
    if name == "resolve_kernel":         # first occurrence and row in, the firsts' unique index, row and unique index out
        return 8 * nnz + 4 * U + 8 * nnz
    if name == "route_kernel":
        return 8 * B + 2 * 5 * nnz + 8 * nnz + 4 * B * (S + 1)
    if name == "shard_partials_kernel":
        return 4 * B * (S + 1) + 4 * nnz + row * U + 4 * S * B * (k + 4)
    if name == "pool_kernel":
        return 4 * (B * F + 1) + 4 * nnz + 4 * k * U + 4 * B * F * k
    if name == "single_gather_kernel":   # rows + shards in, every unique row once, pooled + bag tails out
        return 4 * (B * F + 1) + 5 * nnz + row * U + 4 * B * F * k + 8 * B * F
    if name == "field_partials_kernel":   # pooled vectors and bag tails in, per-shard partials out
        return 4 * B * F * k + 8 * B * F + 4 * S * B * (k + 4)
    if name == "fused_finish_kernel":
        return 4 * B * F * k + 8 * B * F + 4 * B * (k + 4)
    if name == "aggregate_small_kernel":
        return 4 * S * B * (k + 4) + 4 * B * (k + 4)
    if name == "make_dest_kernel":
        return 8 * nnz + 4 * U
    if name == "grad_scatter_kernel":
        # offsets, one index word per occurrence, gE once, A, gL / gF, and every key's summed gradient landing once
        # (the read-modify-write of the gradient rows by the atomics and the per-bag counts of the counted keys are
        # implementation traffic, not algorithmic bytes)
        return 4 * (B * F + 1) + 4 * nnz + (4 * B * F * k if pool else 0) + 4 * B * (k + 4) + 8 * B + row * (U + R)
    if name == "super_dense_kernel":
        return 64 * B * F + (4 * B * F * k if pool else 0) + 4 * B * (k + 4) + 8 * B
    if name == "sample_count_kernel":
        return 4 * (nnz >> st["shift"]) + 4 * U
    if name == "hot_reduce_kernel":
        return 2 * row * R
    if name == "update_rows_kernel":
        return U * (2 * row + 2 * row * (1 + state) + 8)
    if name == "cvt_bf16_kernel":          # one launch per step: gZ and pooled of the backward (the forward's copy of
        return 6 * (B * F * k + B * st["H"])   # pooled comes out of the pooling kernel)
    return None


# Bytes the load / store units move per launch when every occurrence reads (or adds to) its own row: the figure
# the L1 data path sees.  L1 peak = 128 bytes per clock and SM (148 SMs at the sampled SM clock).
def occurrence_bytes(name, st):
    nnz, k = st["nnz"], st["k"]
    if name == "pool_kernel":
        return 4 * k * nnz
    if name in ("shard_partials_kernel", "single_gather_kernel"):
        return (4 * k + 32) * nnz          # the vector and the 32-byte sector that holds the row's tail
    return None


def shift_of(nnz):
    """log2 of the sampling stride of the backward's hot-key count (about 2^20 samples)."""
    shift = 0
    while shift < 6 and (nnz >> shift) > (1 << 20):
        shift += 1
    return shift


def kernel_flops(name, st):
    """Dense flops of one launch (tensor-core GEMMs of the row-split first layer)."""
    if name in ("tc_gemm_fwd", "tc_gemm_dgrad", "tc_gemm_wgrad"):
        return 2 * st["B"] * st["F"] * st["k"] * st["H"]
    return None


# What ncu shows to be the busiest unit of each occurrence-level kernel (captures summarised under profiles/): none of
# them is near the HBM bound of its algorithmic bytes, because every occurrence moves a row through the L1 data path
# while only the unique rows come from HBM.
BOUND_NOTES = {
    "grad_scatter_kernel": "busiest unit per ncu: L1TEX 87 % / L2 67 % (one 16-byte vector atomic per lane and occurrence); DRAM 26 %",
    "shard_partials_kernel": "busiest unit per ncu: L1TEX 73 % (a 272-byte row per occurrence through L1); DRAM 15 %",
    "pool_kernel": "busiest unit per ncu: L1TEX 77 % (a 256-byte vector per occurrence through L1); DRAM 27 %",
    "single_gather_kernel": "busiest unit per ncu: L1TEX 65 % (a 272-byte row per occurrence through L1); DRAM 16 %",
    "update_rows_kernel": "random 272-byte rows of weights and state: DRAM-bound (56 % on a small table under ncu)",
}
TRAFFIC_SOURCE = ("ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch on the benchmark's own batch with a "
                  "4e6-key table (the 2e8-key table cannot be captured under multi-pass replay); constant, not measured "
                  "in this run")


def build_table(w, cfg_index, batches, steps_total, prepop, dev):
    """Table sized for the workload and the number of steps that will run on it; pre-populated (untimed)."""
    import torch
    from paper_1909_04823_b200.binding import DeviceBatch, Table
    max_nnz = int(max(b.nnz for b in batches) * 1.02) + 1024
    if cfg_index == 4:
        max_rows = int(prepop + (steps_total + 2) * batches[0].nnz * w.p_new * 1.3) + 100000
    elif cfg_index == 5:
        max_rows = prepop
    else:
        max_rows = int(sum(len(np.unique(b.ids)) for b in batches) * (3 + steps_total)) + 100000
        max_rows = min(max_rows, 40_000_000)
    uniq0 = int(len(np.unique(batches[0].ids)))
    max_uniq = min(max_nnz, int(uniq0 * 1.5) + 4096)
    t = Table.for_workload(w, max_rows=max_rows, max_nnz=max(max_nnz, w.batch * w.fields), max_batch=w.batch,
                           rows_per_shard=rows_per_shard(w, max_rows), max_uniq=max_uniq)
    if w.hidden:
        t.dense1_set(torch.from_numpy(synth.dense1_weights(w)).to(dev))
    if prepop:
        t0 = time.time()
        per_call = w.batch * w.fields
        stream = synth.Stream(w)
        for ids in stream.prepopulation_ids(chunk=per_call * 8):
            d_all = torch.from_numpy(ids.view(np.int64)).to(dev)
            for lo in range(0, ids.size, per_call):
                n = min(per_call, ids.size - lo)
                pb = synth.prepopulation_batch(ids[lo:lo + n], w.fields)
                t.find_or_insert(DeviceBatch(pb.offsets, d_all[lo:lo + n], None, pb.batch, dev), True)
        t.check_status()
        log(f"[bench] pre-populated {sum(t.size())} keys in {time.time() - t0:.1f}s")
    return t


def run_workload(args, cfg_index, w, ctx, *, steps, warmup, repeats, modes, want_e2e, want_cpu, profile_in_timed):
    """Measures one workload.  modes: "eager" and / or "graph".  Returns a dict with one entry per mode
    (step times of every repeat, per-kernel shares, dominant-kernel roofline) plus e2e / cpu_baseline."""
    import torch
    import torch.distributed as dist
    from paper_1909_04823_b200.binding import DeviceBatch

    rank, world, dev, sampler = ctx["rank"], ctx["world"], ctx["dev"], ctx["sampler"]
    hbm_peak, tc_peak, peak_kind = ctx["peaks"]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    prepop = w.prepopulate
    if cfg_index == 5:
        free_b, _ = torch.cuda.mem_get_info()
        vocab = w.vocab
        if args.vocab:
            prepop = vocab = args.vocab
        per_key = 2 * (4 * w.emb_dim + 16) * 1.06 + 16 * 2.2      # rows + state + slots at load 0.5
        fit = int((free_b - 14e9) / per_key)
        if fit < prepop:
            prepop = vocab = max(1_000_000, (fit // 1_000_000) * 1_000_000)
            log(f"[bench] only {free_b / 1e9:.0f} GB free: table scaled to {prepop} keys")
        w = w.scaled(vocab=vocab, prepopulate=prepop)
    stream = synth.Stream(w)
    steps_total = (steps * repeats + warmup + 3) * len(modes) + (steps if "graph" in modes else 0) + 16
    n_batches = 2 if cfg_index != 4 else min(steps + warmup, 12)
    t0 = time.time()
    batches = [stream.next_batch() for _ in range(n_batches)]
    log(f"[bench] generated {n_batches} batches of {w.name}: nnz {batches[0].nnz} in {time.time() - t0:.1f}s")
    t = build_table(w, cfg_index, batches, steps_total, prepop, dev)

    B, F, k, S, H = w.batch, w.fields, w.emb_dim, w.shards, w.hidden
    dbs = [DeviceBatch.from_synth(b, dev) for b in batches]
    g_host = synth.upstream_grads(w, B, 0)
    gd = {n_: torch.from_numpy(v).to(dev) for n_, v in g_host.items()}
    small = bool(w.ops & (OP_LR | OP_FM)); pool = bool(w.ops & (OP_POOL | OP_DENSE1))
    part_small = torch.zeros((S, B, k + 4), device=dev) if small else None
    pooled = torch.zeros((B, F * k), device=dev) if pool else None
    out_small = torch.zeros((B, k + 4), device=dev)
    Z = torch.zeros((B, H), device=dev) if H else None
    gE_work = torch.zeros((B, F * k), device=dev) if (w.ops & OP_DENSE1) else None
    gE = gd.get("gE") if (w.ops & OP_POOL) else None
    gZ = gd.get("gZ") if (w.ops & OP_DENSE1) else None

    # closed loop: the upstream gradients of every step come from the fixed read-out applied to that step's own
    # forward results (labels and continuous features are seeded and resident on the device)
    closed = None
    if args.closed_loop:
        n_dense = 13 if cfg_index == 2 else 0          # the Criteo shape: 13 continuous columns beside the 26 categorical
        hc = synth.head_constants(w, n_dense)
        closed = dict(hc={n_: (torch.from_numpy(v).to(dev) if isinstance(v, np.ndarray) and v.ndim else v) for n_, v in hc.items()},
                      y=torch.from_numpy(synth.labels(w, B, 0)).to(dev),
                      xd=torch.from_numpy(synth.dense_features(w, B, 0, n_dense)).to(dev) if n_dense else None,
                      logit=torch.zeros(B, device=dev), loss=torch.zeros(B, device=dev),
                      gL=torch.zeros(B, device=dev), gF=torch.zeros(B, device=dev),
                      gE=torch.zeros((B, F * k), device=dev) if (pool and not (w.ops & OP_DENSE1)) else None,
                      gZ=torch.zeros((B, H), device=dev) if (w.ops & OP_DENSE1) else None)

    def step(i):
        db = dbs[i % len(dbs)]
        t.find_or_insert(db, True)
        if args.fused or args.fused_partials:
            t.forward_fused(w.ops | (16 if args.fused_partials else 0), db, None, pooled, out_small, Z)
        else:
            t.forward_partials(w.ops, db, part_small, pooled)
            t.aggregate(w.ops, db, part_small, pooled, out_small=out_small, Z=Z)
        if closed is None:
            t.backward_update(w.ops, db, out_small, pooled, Z, gd.get("gL"), gd.get("gF"), gE, gZ, gE_work)
        else:
            c = closed
            t.head(w.ops, B, c["hc"], out_small, pooled, Z, c["xd"], c["y"], c["logit"], c["loss"], c["gL"], c["gF"],
                   c["gE"], c["gZ"])
            t.backward_update(w.ops, db, out_small, pooled, Z, c["gL"], c["gF"], c["gE"], c["gZ"], gE_work)

    U = None
    stats = None

    def kernel_table(prof, n_steps):
        per = {}
        for name, ms in prof:
            a = per.setdefault(name, [0, 0.0]); a[0] += 1; a[1] += ms
        tot_k = sum(v[1] for v in per.values()) or 1.0
        kernels = []
        for name, (n_, ms) in sorted(per.items(), key=lambda kv: -kv[1][1]):
            by = kernel_bytes(name, stats)
            fl = kernel_flops(name, stats)
            avg = ms / n_
            ob = occurrence_bytes(name, stats)
            kernels.append({"kernel": name, "launches": n_, "ms_per_launch": round(avg, 4), "share": round(ms / tot_k, 4),
                            "alg_gbs": None if by is None else round(by / avg / 1e6, 1),
                            "tflops": None if fl is None else round(fl / avg / 1e9, 1),
                            # occurrence-level bytes through L1 against 128 B / clock / SM x 148 SMs x 1.965 GHz
                            "l1_gbs": None if ob is None else round(ob / avg / 1e6, 1),
                            "l1_frac_of_nominal": None if ob is None else round(ob / avg / 1e6 / (128 * 148 * 1.965), 3)})
        roofline = None
        for top in kernels:      # the kernel with the largest share of the timed region that has a byte / flop model
            if top["alg_gbs"] is not None:
                tr = NCU_DRAM_TRAFFIC.get((w.name.split("_")[0], top["kernel"]))
                roofline = {"bound": "hbm", "kernel": top["kernel"], "achieved": top["alg_gbs"], "peak": hbm_peak,
                            "unit": "GB/s", "frac": round(top["alg_gbs"] / hbm_peak, 4), "traffic": tr,
                            "traffic_source": TRAFFIC_SOURCE if tr is not None else None,
                            "peak_kind": f"of {peak_kind}", "ms_per_launch": top["ms_per_launch"], "share": top["share"],
                            "note": BOUND_NOTES.get(top["kernel"])}
                break
            if top["tflops"] is not None:
                roofline = {"bound": "tensor", "kernel": top["kernel"], "achieved": top["tflops"], "peak": tc_peak,
                            "unit": "TFLOP/s", "frac": round(top["tflops"] / tc_peak, 4), "traffic": None,
                            "peak_kind": f"of {peak_kind} (sustained bf16)", "ms_per_launch": top["ms_per_launch"],
                            "share": top["share"]}
                break
        step_bytes = sum((kernel_bytes(kk["kernel"], stats) or 0) * kk["launches"] for kk in kernels) / max(1, n_steps)
        return kernels, roofline, step_bytes

    results = {}
    windows = []
    done_steps = 0
    for i in range(warmup):
        step(i)
    done_steps += warmup
    t.check_status()
    barrier()
    U = int(dbs[0].n_uniq.item())
    stats = dict(nnz=batches[0].nnz, B=B, F=F, k=k, S=S, H=H, U=U, ops=w.ops,
                 adagrad=(w.optimizer == synth.OPT_ADAGRAD), rep_rows=0,
                 super=(k > 28 and batches[0].nnz >= (1 << 20) and batches[0].vals is None),
                 shift=shift_of(batches[0].nnz), new_keys=(w.p_new > 0 or not w.prepopulate))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for mode in modes:
        graphs = None
        if mode == "graph":
            graphs = []                       # one graph per batch; the step has no host synchronisation and allocates nothing
            for i in range(len(dbs)):
                gph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gph):
                    step(i)
                graphs.append(gph)
            for i in range(max(warmup, 3)):
                graphs[i % len(graphs)].replay()
            barrier()
        prof_live = graphs is None and profile_in_timed
        launches0 = t.launch_count()
        if prof_live:
            t.profile_enable(True)
        rep_ms, rep_clk, prof = [], [], []
        for r in range(repeats):
            barrier()
            h0 = time.perf_counter()
            e0.record()
            for i in range(steps):
                if graphs is None:
                    step(done_steps + i)
                else:
                    graphs[(done_steps + i) % len(graphs)].replay()
            e1.record()
            barrier()
            h1 = time.perf_counter()
            done_steps += steps
            rep_ms.append(max_over_ranks(e0.elapsed_time(e1), world, dev) / steps)
            windows.append((h0, h1))
            if sampler:
                rep_clk.append(sampler.window(h0, h1))
            if prof_live:
                prof += t.profile_read()
        n_prof_steps = steps * repeats
        if not prof_live:
            # kernel shares from an eager pass outside the timed region; launches per step counted there too
            t.profile_enable(True)
            launches0 = t.launch_count()
            for i in range(steps):
                step(done_steps + i)
            done_steps += steps
            barrier()
            prof = t.profile_read()
            n_prof_steps = steps
        t.profile_enable(False)
        launches = (t.launch_count() - launches0) // max(1, (repeats if prof_live else 1))
        t.check_status()
        kernels, roofline, step_bytes = kernel_table(prof, n_prof_steps)
        ms_step = float(np.median(rep_ms))
        results[mode] = {"ms_per_step": ms_step, "value": job_throughput(B, world, ms_step),
                         "repeats": {"n": repeats, "steps_each": steps, "ms_per_step": [round(v, 4) for v in rep_ms],
                                     "min": round(min(rep_ms), 4), "max": round(max(rep_ms), 4),
                                     "sm_mhz": [c["sm_mhz"] for c in rep_clk],
                                     "reasons": sorted({r_ for c in rep_clk for r_ in c["reasons"]})},
                         "kernels": kernels, "roofline": roofline, "step_bytes": step_bytes, "gpu_launches": int(launches)}

    # ---- end to end from pinned host buffers
    e2e = None
    if want_e2e:
        try:
            hb = batches[0]
            h_off = torch.from_numpy(hb.offsets).pin_memory()
            h_ids = torch.from_numpy(hb.ids.view(np.int64)).pin_memory()
            h_out = [torch.empty((B, k + 4), dtype=torch.float32).pin_memory() for _ in range(2)]
            kw = dict(d_pooled=pooled, d_Z=Z, gL=gd.get("gL"), gF=gd.get("gF"), gE=gE, gZ=gZ, gE_work=gE_work)

            def run_blocking(n):
                for i in range(n):
                    t.step_host(w.ops, B, hb.nnz, h_off, h_ids, None, h_out[i & 1], **kw)

            def run_pipelined(n):          # the copy of step i+1 overlaps the kernels of step i
                prev = None
                for i in range(n):
                    tk = t.step_host_submit(w.ops, B, hb.nnz, h_off, h_ids, None, h_out[i & 1], **kw)
                    if prev is not None:
                        t.step_host_wait(prev)
                    prev = tk
                t.step_host_wait(prev)

            n_e2e = max(3, min(steps, 10))
            ms_mode = {}
            for name, fn in (("blocking", run_blocking), ("pipelined", run_pipelined)):
                fn(max(1, min(warmup, 3)))
                barrier()
                e0.record()
                fn(n_e2e)
                e1.record()
                barrier()
                ms_mode[name] = max_over_ranks(e0.elapsed_time(e1) / n_e2e, world, dev)
            ms_e = ms_mode["pipelined"]
            e2e = {"value": job_throughput(B, world, ms_e), "unit": UNIT, "ms_per_step": ms_e,
                   "mode": "des_step_host_submit / des_step_host_wait from pinned host buffers, two steps in flight; "
                           "copied every step: offsets + ids host to device, out_small [B][k+4] back; resident on the "
                           "device: the upstream gradients gL / gF / gE (they come from the rest of the model) and the "
                           "pooled output (its consumer)",
                   "blocking_ms_per_step": ms_mode["blocking"],
                   "h2d_bytes_per_step": int(h_off.numel() * 4 + h_ids.numel() * 8),
                   "d2h_bytes_per_step": int(h_out[0].numel() * 4)}
        except Exception as ex:  # keep the device-resident number even if the host path fails
            log(f"[bench] e2e failed: {ex!r}")
        t.check_status()

    # ---- CPU oracle on a bounded sample (rank 0, single GPU runs only): one core, then all cores
    cpu = None
    if want_cpu:
        try:
            import oracle
            v, bs, sec = time_oracle(w, batches[0], g_host, budget_s=args.cpu_budget * 0.6)
            cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                   "sample": f"first {bs} of {B} samples of one batch ({sec:.1f} s), table holding the keys it touches"}
            try:
                n_thr = oracle.num_threads(True)
                v2, bs2, sec2 = time_oracle(w, batches[0], g_host, budget_s=args.cpu_budget * 0.4, omp=True)
                cpu["all_cores"] = {"value": v2, "unit": UNIT, "cores": n_thr, "host_cpus": os.cpu_count(),
                                    "kind": "oracle, same source built with -fopenmp",
                                    "sample": f"first {bs2} of {B} samples of one batch ({sec2:.1f} s)"}
            except Exception as ex:
                log(f"[bench] all-cores cpu baseline failed: {ex!r}")
        except Exception as ex:
            log(f"[bench] cpu baseline failed: {ex!r}")

    table_keys = sum(t.size())
    t.close()
    del t
    torch.cuda.empty_cache()
    return dict(w=w, results=results, e2e=e2e, cpu=cpu, windows=windows, nnz=batches[0].nnz, U=U, table_keys=table_keys,
                l2_note="inputs larger than L2 (no flush)" if batches[0].nnz * 8 > 126e6 else
                        "small workload: inputs fit in L2, two batches alternate, no flush")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--repeats", type=int, default=5, help="the --steps region is timed this many times back to back")
    ap.add_argument("--config", type=int, default=5, help="workload 1..5 (default: 5, the large multi-hot one)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--vocab", type=int, default=0, help="override the number of pre-populated keys (config 5)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-side-configs", action="store_true",
                    help="skip the short eager / graph-replay runs of the other four workloads")
    ap.add_argument("--graph", action="store_true",
                    help="replay the step from a CUDA graph (launch-bound small workloads); per-kernel times then "
                         "come from a separate, untimed eager pass")
    ap.add_argument("--fused", action="store_true",
                    help="use des_forward_fused (per-shard partials kept on chip) instead of partials + aggregate")
    ap.add_argument("--fused-partials", action="store_true",
                    help="des_forward_fused in its shard-by-shard form: per-shard partials formed on chip in shard order, "
                         "aggregated and passed through F without being written (bit-identical to the default path)")
    ap.add_argument("--closed-loop", action="store_true",
                    help="gradients from the fixed read-out (des_head) on the step's own forward instead of seeded "
                         "upstream gradients: the whole Criteo-shaped Wide&Deep / DeepFM step with --config 2 / 3 "
                         "(throughput only: the dataset is not available here)")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    args.repeats = max(args.repeats, 1)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    w = synth.config(args.config)
    w = per_rank_workload(w, rank, world)           # every replica has its own data stream

    # ------------------------------------------------------------------ reference arm: the CPU oracle
    if args.impl == "reference":
        if rank != 0:
            return 0
        # the sample touches a few thousand keys; their rows are a pure function of the id, so the oracle
        # needs no pre-populated table to reproduce the first step of the full workload
        st = synth.Stream(w)
        b = st.next_batch()
        g = synth.upstream_grads(w, b.batch, 0)
        budget = min(args.cpu_budget, 120.0 / max(1, args.steps + args.warmup))
        v, bs, sec = time_oracle(w, b, g, budget_s=budget, steps=max(1, args.steps), warmup=args.warmup)
        line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": {"workload": w.name, "batch": w.batch, "fields": w.fields, "emb_dim": w.emb_dim,
                           "shards": w.shards, "sample": f"first {bs} of {w.batch} samples per step"},
                "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "host_cpus": os.cpu_count(), "kind": "oracle",
                                 "sample": f"first {bs} of {w.batch} samples of one batch, table holding the keys it touches"},
                "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line), flush=True)
        return 0

    # ------------------------------------------------------------------ our arm
    import torch
    import torch.distributed as dist
    from paper_1909_04823_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the DES path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    sampler = ClockSampler(local) if rank == 0 else None     # every 20 ms, from here to the end of the timed regions
    ctx = dict(rank=rank, world=world, dev=dev, sampler=sampler, peaks=measured_peaks())
    hbm_peak = ctx["peaks"][0]

    # ---- the other workloads, short (single-GPU default run only): eager and CUDA-graph replay
    side = []
    if world == 1 and not args.no_side_configs and args.config == 5 and not args.graph:
        for ci in (1, 2, 3, 4):
            try:
                r = run_workload(args, ci, synth.config(ci), ctx, steps=20 if ci < 4 else 6, warmup=3, repeats=3,
                                 modes=["eager", "graph"], want_e2e=False, want_cpu=False, profile_in_timed=False)
                for mode in ("eager", "graph"):
                    m = r["results"][mode]
                    rf = m["roofline"] or {}
                    side.append({"workload": r["w"].name, "launch": mode, "ms_per_step": round(m["ms_per_step"], 4),
                                 "value": round(m["value"], 1), "unit": UNIT, "repeats_ms": m["repeats"]["ms_per_step"],
                                 "nnz_per_step": r["nnz"], "unique_keys_per_step": r["U"],
                                 "dominant_kernel": rf.get("kernel"), "dominant_share": rf.get("share"),
                                 "dominant_achieved": rf.get("achieved"), "dominant_unit": rf.get("unit"),
                                 "dominant_frac": rf.get("frac"), "gpu_launches_per_step": m["gpu_launches"] // max(1, 20 if ci < 4 else 6)})
            except Exception as ex:
                log(f"[bench] side run of config {ci} failed: {ex!r}")
                side.append({"workload": f"config {ci}", "error": repr(ex)})

    mode = "graph" if args.graph else "eager"
    # (the default run also replays the same step from a CUDA graph, reported beside the eager headline)
    modes = [mode] if (args.graph or world > 1) else ["eager", "graph"]
    r = run_workload(args, args.config, w, ctx, steps=args.steps, warmup=args.warmup, repeats=args.repeats, modes=modes,
                     want_e2e=not (args.no_e2e or args.closed_loop), want_cpu=(rank == 0 and world == 1 and not args.no_cpu_baseline),
                     profile_in_timed=True)
    clocks = sampler.stop(r["windows"]) if sampler else None
    m = r["results"][mode]
    w = r["w"]
    ms_step = m["ms_per_step"]
    B, F, k, S = w.batch, w.fields, w.emb_dim, w.shards
    step_bytes = m["step_bytes"]
    row_b = 4 * k + 16
    extra = max(0, r["nnz"] - r["U"])                    # occurrences beyond the first of their key
    occ_bytes = step_bytes + extra * ((row_b if (w.ops & (OP_LR | OP_FM)) else 0)
                                      + (4 * k if (w.ops & (OP_POOL | OP_DENSE1)) else 0) + row_b)
    if rank == 0:
        line = {"metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name, "batch": B, "fields": F, "emb_dim": k, "shards": S,
                           "nnz_per_step": r["nnz"], "unique_keys_per_step": r["U"], "table_keys": r["table_keys"],
                           "ops": w.ops, "optimizer": "adagrad" if w.optimizer else "sgd",
                           "parallelism": f"replicas x{world}" if world > 1 else "1 GPU",
                           "launch": "CUDA graph replay" if args.graph else "eager",
                           "forward": "fused, single gather (per-shard partials never formed)" if args.fused else
                                      "fused, per-shard partials formed on chip in shard order" if args.fused_partials else
                                      "per-shard partials materialised, then aggregated",
                           "tensor_core_gemm": bool(binding.uses_tensor_cores()),
                           "gradients": "closed loop: fixed read-out + log loss on the step's own forward (synthetic labels; "
                                        "the paper's datasets are not available here)" if args.closed_loop else
                                        "seeded upstream gradients, resident on the device",
                           "l2": r["l2_note"]},
                "timing": "ms_per_step = median over `repeats.n` back-to-back timings of --steps steps each",
                "repeats": m["repeats"],
                "clocks": clocks, "e2e": r["e2e"], "gpu_launches": int(m["gpu_launches"]),
                "roofline": m["roofline"],
                "hbm": {"alg_bytes_per_step": int(step_bytes), "alg_gbs": round(step_bytes / ms_step / 1e6, 1),
                        "frac_of_measured_copy": round(step_bytes / ms_step / 1e6 / hbm_peak, 4),
                        "frac_of_nominal_8000": round(step_bytes / ms_step / 1e6 / 8000.0, 4),
                        # occurrence-level accounting: what the load / store units move when every occurrence
                        # gathers (twice: per-shard partials and pooling) and scatters its own row; these are
                        # mostly L1 / L2 hits in a skewed batch, so this is not an HBM figure
                        "occ_bytes_per_step": int(occ_bytes), "occ_gbs": round(occ_bytes / ms_step / 1e6, 1)},
                "kernels": m["kernels"], "cpu_baseline": r["cpu"], "configs": side}
        if "graph" in r["results"] and mode != "graph":
            gm = r["results"]["graph"]
            line["graph_replay"] = {"ms_per_step": gm["ms_per_step"], "value": gm["value"], "unit": UNIT,
                                    "repeats_ms": gm["repeats"]["ms_per_step"],
                                    "note": "the same step replayed from a CUDA graph (one graph per resident batch)"}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
