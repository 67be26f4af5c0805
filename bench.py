#!/usr/bin/env python
"""Benchmark of the ROBE-Z hot path on B200.

One step = one pass of the whole path over one batch: robe_forward (hash -> offset -> circular
block gather -> bag sum-pool) followed by robe_backward (block scatter-add of the output
gradient with the SGD step fused in) - called as robe_forward_keep / robe_backward_kept when
the backward sorts the blocks, so that every id is hashed once per step.  The default workload is the multi-hot pooled
configuration whose 1 GB array does not fit in L2 (26 tables, d=64, Z=16, batch 16384, bags of
about 20 ids).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

prints ONE JSON line.  With N > 1 (launched by torch.distributed.run) every rank runs its own
batch shard on its own replica of the array (weak scaling, no data-path collective) and rank 0
reports the aggregate with the time taken as the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2108_02191_b200 import synth  # noqa: E402

METRIC = "robe_lookups_per_s_fwd_bwd"
UNIT = "ids/s"

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) recorded from one-pass ncu
# captures of the full-size workload; the summaries under profiles/ hold the commands.  A record
# applies only to the exact configuration it was captured on (workload, backward variant, shared
# block starts, id type, bag layout, workload's own batch): any other run reports traffic = null.
# Records go stale when a kernel changes: they are re-captured with the kernel, never edited.
NCU_TRAFFIC_RECORDS = {
    # (workload, backward variant, block starts shared, id type, bag layout)
    ("cfg4_multihot", "binned", True, "int64", "sample-major"): {
        "forward": 4_412_000_000, "backward": 4_838_700_000,
        "source": "profiles/launches_cfg4_multihot.md: full-size one-pass ncu capture of `python bench.py --steps 3 "
                  "--warmup 3 --no-cpu-baseline`; forward = fwd_staged_kernel, backward = sort_count + sort_scan + "
                  "sort_scatter + binned_apply"},
    ("cfg4_multihot", "atomic", False, "int64", "sample-major"): {
        "forward": 4_130_800_000, "backward": 7_378_600_000,
        "source": "profiles/launches_cfg4_multihot.md: full-size one-pass ncu capture of `python bench.py --steps 3 "
                  "--warmup 3 --no-cpu-baseline --backward atomic`"},
    ("cfg4_multihot", "det", True, "int64", "sample-major"): {
        "forward": 4_411_800_000, "backward": 7_246_000_000,
        "source": "profiles/launches_cfg4_multihot.md: full-size one-pass ncu capture of `python bench.py --steps 3 "
                  "--warmup 3 --no-cpu-baseline --backward det`; backward = 4 sort passes, window bounds and classes, "
                  "apply kernels"},
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def algorithmic_bytes(w, nbags, nnz, bags, id_bytes=8):
    """Bytes the method itself must move per launch (useful-bytes model):
    forward  = 8 (4 with int32 ids) per id (index) + d*s_a per id (array elements read) + 8 per bag (offset, pooled
               only) + 4d per bag (output row written);
    backward = 8 per id + 2*4d per id (read-modify-write of the slots) + 8 per bag (pooled only)
               + 4d per bag (gradient row read once)."""
    s_a = 4 if w.array_dtype == "f32" else 2
    off = 8 * (nbags + 1) if bags else 0
    fwd = id_bytes * nnz + w.d * s_a * nnz + off + 4 * w.d * nbags
    bwd = id_bytes * nnz + 2 * 4 * w.d * nnz + off + 4 * w.d * nbags
    return fwd, bwd


def forward_byte_models(w, nbags, nnz, bags, id_bytes=8):
    """The forward's bytes per launch under the three models the results are read against:
    useful       what the method itself must move (algorithmic_bytes);
    sector       the same with the array counted in 32-byte sectors: a Z-element block at an
                 arbitrary element offset covers 1 + (Z-1)/E sectors on average (E elements per
                 sector) - the paper's Table 1 restated for sectors;
    l2_resident  ids, offsets and output only: the floor when the array is served from L2."""
    s_a = 4 if w.array_dtype == "f32" else 2
    zb = min(w.Z, w.d)
    e_per_sector = 32 // s_a
    blocks = -(-w.d // zb)
    rest = id_bytes * nnz + (8 * (nbags + 1) if bags else 0) + 4 * w.d * nbags
    return {"useful": rest + w.d * s_a * nnz,
            "sector": rest + blocks * (1 + (zb - 1) / e_per_sector) * 32 * nnz,
            "l2_resident": rest}


class ClockSampler:
    """SM clock and throttle-reason samples taken while the timed region runs.

    Reads (never sets) the clocks: through NVML in a background thread, every 2 ms, so that even a
    40 ms timed region yields a dozen samples; if NVML cannot be loaded, through `nvidia-smi -lms`,
    whose loop delivers a sample every 10-15 ms.  stop(window) keeps the samples taken inside the
    timed region (the sampler is started before the warm-up so that it is delivering by then)."""

    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    PERIOD_S = 0.002

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None
        self.thread = None
        self.samples = []   # (time.time(), sm_mhz, reasons bit mask)
        self.max_mhz = None
        self._stop = False

    def _nvml_loop(self, nvml, handle):
        reasons_of = getattr(nvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            nvml.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop:
            try:
                mhz = nvml.nvmlDeviceGetClockInfo(handle, nvml.NVML_CLOCK_SM)
                mask = reasons_of(handle)
                self.samples.append((time.time(), float(mhz), int(mask)))
            except Exception:
                pass
            time.sleep(self.PERIOD_S)

    def start(self):
        try:
            import threading

            import pynvml as nvml
            nvml.nvmlInit()
            handle = nvml.nvmlDeviceGetHandleByIndex(self.gpu)
            self.max_mhz = float(nvml.nvmlDeviceGetMaxClockInfo(handle, nvml.NVML_CLOCK_SM))
            self.nvml = nvml
            self.thread = threading.Thread(target=self._nvml_loop, args=(nvml, handle), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "10",
                 "-i", str(self.gpu)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def _stamp(text):
        """Seconds since the epoch of an nvidia-smi timestamp (local time, milliseconds)."""
        import datetime
        return datetime.datetime.strptime(text, "%Y/%m/%d %H:%M:%S.%f").timestamp()

    def stop(self, window=None):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.thread is not None:
            self._stop = True
            self.thread.join(timeout=2)
            nvml = self.nvml
            names = {"hw_slowdown": "HwSlowdown", "hw_thermal_slowdown": "HwThermalSlowdown",
                     "sw_thermal_slowdown": "SwThermalSlowdown", "sw_power_cap": "SwPowerCap"}
            bits = {k: getattr(nvml, "nvmlClocksEventReason" + v, None) or getattr(nvml, "nvmlClocksThrottleReason" + v)
                    for k, v in names.items()}
            kept = [smp for smp in self.samples if window is None or window[0] <= smp[0] <= window[1]]
            if kept:
                out["sm_mhz"] = float(np.median([smp[1] for smp in kept]))
                out["sm_max_mhz"] = self.max_mhz
                out["samples"] = len(kept)
                out["reasons"] = sorted(k for k, bit in bits.items() if any(smp[2] & bit for smp in kept))
            out["source"] = "nvml"
            try:
                nvml.nvmlShutdown()
            except Exception:
                pass
            return out
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    if window is not None:
                        ts = self._stamp(f[0])
                        if ts < window[0] or ts > window[1]:
                            continue
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["sm_max_mhz"] = float(max(mx))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        out["source"] = "nvidia-smi"
        return out


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def rank_batch_variants(rank: int, nb: int):
    """Seeds of the id batches of one rank: every rank draws its own shard of the global batch
    (data parallel by sample), so no two ranks ever share a variant number."""
    return [1000 * rank + v for v in range(nb)]


def aggregate_over_ranks(dist, device, times_ms, units):
    """Whole-job figures from per-rank ones: every time becomes the MAXIMUM over ranks, the units
    of work (ids) the SUM over ranks.  `dist` is torch.distributed or None for one process; the
    reductions are the only communication of the benchmark (the data path has none)."""
    t = torch.tensor([float(v) for v in times_ms], dtype=torch.float64, device=device)
    u = torch.tensor([float(v) for v in units], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return [float(v) for v in t.tolist()], [float(v) for v in u.tolist()]


WORKLOAD_HELP = ("cfg2 | cfg3_z<Z> | cfg4 | cfg5_<1m|100m|10g>_z<Z>[_bf16]  (cfg5 = cfg5_100m_z32); "
                 "cfg4 is the headline workload, the others are the parity-test shapes")


def pick_workload(name: str):
    """A workload by name, see WORKLOAD_HELP."""
    if name == "cfg2":
        return synth.workload(2)
    if name == "cfg4":
        return synth.workload(4)
    if name == "cfg5":
        return synth.workload(5)
    parts = name.split("_")
    if parts[0] == "cfg3" and len(parts) == 2 and parts[1].startswith("z"):
        return synth.workload(3, Z=int(parts[1][1:])).with_(name=name)
    if parts[0] == "cfg5" and len(parts) in (3, 4) and parts[2].startswith("z"):
        M = {"1m": 262_144, "100m": 25_000_000, "10g": 2_500_000_000}[parts[1]]
        kw = dict(M=M, Z=int(parts[2][1:]))
        if len(parts) == 4:
            if parts[3] != "bf16":
                raise ValueError(name)
            kw["array_dtype"] = "bf16"
        w = synth.workload(5, **kw)
        return w.with_(name=name)
    raise ValueError(f"unknown workload {name!r}: {WORKLOAD_HELP}")


# -------------------------------------------------------------------------------------------
# reference arm / cpu baseline: the oracle as it stands, on the host cores
# -------------------------------------------------------------------------------------------

def oracle_step_rate(w, sample_batch: int, array_h=None, variant=0):
    """Times oracle forward + fp64 backward on `sample_batch` samples of workload w.
    Returns (ids per second, ids in the sample, threads used, seconds)."""
    from oracle import robe_oracle as orc
    ids, offs = synth.make_ids(w, sample_batch, variant)
    grad = synth.make_grad_out(w, sample_batch, variant)
    if array_h is None:
        array_h = synth.array_to_numpy(synth.make_array(w, "cpu"))
    o = orc.Oracle(w.M, w.Z, w.d, w.num_tables, orc.hash_constants(w.hash_seed))
    t0 = time.perf_counter()
    o.forward(array_h, ids, offs, sample_batch)
    o.backward_f64(grad, ids, offs, sample_batch)
    dt = time.perf_counter() - t0
    return len(ids) / dt, len(ids), orc.num_threads(), dt


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    array_h = synth.array_to_numpy(synth.make_array(w, "cpu"))
    # Every step runs the oracle on the workload's whole batch - the sample the cpu_baseline leg of
    # the other arm times - unless the first (warm-up) step shows that steps + warmup such steps
    # would take more than about three minutes; then the batch is cut by a power of two.
    sample_batch = w.batch
    _, _, _, t_full = oracle_step_rate(w, sample_batch, array_h, variant=0)
    planned = (args.steps + args.warmup) * t_full
    while planned > 200.0 and sample_batch > 64:
        sample_batch //= 2
        planned /= 2
    for i in range(1, args.warmup):
        oracle_step_rate(w, sample_batch, array_h, variant=i)
    total_ids, total_t, threads = 0, 0.0, 1
    for i in range(args.steps):
        rate, n, threads, dt = oracle_step_rate(w, sample_batch, array_h, variant=100 + i)
        total_ids += n
        total_t += dt
    value = total_ids / total_t
    sample = f"{sample_batch} of {w.batch} samples per step (forward + fp64 backward)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# -------------------------------------------------------------------------------------------
# our arm
# -------------------------------------------------------------------------------------------

def run_ours(args, w):
    import paper_2108_02191_b200 as robe

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    else:
        dist = None

    NB = 4  # distinct pre-generated id batches, rotated so ids are never L2-warm
    bags = w.bag_rule is not None
    B, T, d = w.batch, w.num_tables, w.d
    nbags = B * T
    batches = []
    table_major = args.bag_layout == "table-major"
    for v in rank_batch_variants(rank, NB):
        ids_v = synth.make_ids(w, B, variant=v)
        batches.append(synth.to_table_major(ids_v[0], ids_v[1], B, T) if table_major else ids_v)
    array = synth.make_array(w, dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.data_seed + 17 * rank)
    grad_out = torch.randn(B, T, d, device=dev, dtype=torch.float32, generator=gen)
    out = torch.empty(B, T, d, device=dev, dtype=torch.float32)
    id_dtype = torch.int32 if args.ids == "int32" else torch.int64
    id_bytes = 4 if args.ids == "int32" else 8
    d_ids = [torch.from_numpy(b[0]).to(dev).to(id_dtype) for b in batches]
    d_offs = [None if b[1] is None else torch.from_numpy(b[1]).to(dev) for b in batches]

    h = robe.robe_create(w.M, w.Z, w.d, T, w.hash_seed)
    robe.robe_attach_array(h, array)
    if table_major:
        robe.robe_set_option(h, robe.ROBE_OPT_BAG_LAYOUT, robe.ROBE_BAGS_TABLE_MAJOR)
    robe.robe_set_option(h, robe.ROBE_OPT_FWD_KERNEL, args.fwd_kernel)
    if (args.bwd_kernel == 0 and not bags and w.id_dist.startswith("zipf") and min(w.Z, w.d) >= 64 and d <= 128):
        # skewed ids, long blocks: the repeats of an id are merged in the warp (the caller knows its
        # ids; the library cannot tell from the shapes)
        args.bwd_kernel = 5
    robe.robe_set_option(h, robe.ROBE_OPT_BWD_KERNEL, args.bwd_kernel)
    l2_keep = args.l2_keep
    robe.robe_set_option(h, robe.ROBE_OPT_ARRAY_L2_KEEP, l2_keep)
    lr = 1.0  # the paper trains its DLRM with plain SGD at learning rate 1.0 (Section 5)
    ws = None
    bwd_launches = 1
    if args.backward == "auto":
        # Binned pays when the array lives in HBM and a launch touches each array sector several
        # times (ids per step x d >= array length); else the plain atomic variant is the faster one.
        hbm_resident = w.M * (4 if w.array_dtype == "f32" else 2) > 2 * 126e6
        coverage = float(np.mean([len(b[0]) for b in batches])) * w.d / w.M
        args.backward = "binned" if (hbm_resident and coverage >= 1.0 and w.array_dtype == "f32") else "atomic"
    if args.backward == "binned":
        robe.robe_set_option(h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_BINNED)
        ws = torch.empty(robe.robe_backward_workspace_bytes(h, B, max(len(b[0]) for b in batches)),
                         dtype=torch.uint8, device=dev)
        bwd_launches = (1 if bags else 0) + 5  # (bag numbers,) keys, count, scan, scatter, apply
    # a bf16 array is read-only for the library: its gradient goes to a dense fp32 array instead
    # of the fused SGD step (the array stays as it is)
    dense = torch.zeros(w.M, dtype=torch.float32, device=dev) if w.array_dtype != "f32" else None
    # Data-parallel training step (more than one rank, fp32 array): the replicas must apply the
    # SAME update, so the fused step gives way to backward into a dense gradient -> all-reduce
    # (sum over ranks, 4 M bytes) -> robe_apply_sgd.  One rank needs no exchange and keeps the
    # fused step unless --dp-step on asks for the three-phase step.
    dp_step = w.array_dtype == "f32" and (args.dp_step == "on" or (args.dp_step == "auto" and world > 1))
    if dp_step:
        dense = torch.zeros(w.M, dtype=torch.float32, device=dev)
    if args.backward == "det":
        robe.robe_set_option(h, robe.ROBE_OPT_BWD_MODE, robe.ROBE_BWD_DETERMINISTIC)
        ws = torch.empty(robe.robe_backward_workspace_bytes(h, B, max(len(b[0]) for b in batches)),
                         dtype=torch.uint8, device=dev)
        # keys (+ bag numbers), three kernels per 8-bit sort pass, apply, long walks (when no
        # block is short), low slots (when blocks are longer than one element)
        npass = -(-max(1, (w.M - 1).bit_length()) // 8)
        zb = min(w.Z, w.d)
        bwd_launches = ((1 if bags else 0) + 1 + 3 * npass + 1 + (1 if w.d % zb == 0 else 0)
                        + (1 if zb > 1 else 0))
        # a densely touched array: window bounds, window classes and the window kernel as well
        terms = float(np.mean([len(b[0]) for b in batches])) * w.d
        if w.d % zb == 0 and zb <= 128 and 2 * terms >= w.M:
            bwd_launches += 3
    # One training step hashes every id once: the forward leaves the block starts in the workspace
    # and the sort-based backward takes them from there (rows of up to 128 elements; longer rows
    # use a forward kernel that keeps nothing, and the key kernels then run inside the forward call).
    share_keys = args.share_keys and ws is not None
    if share_keys and w.d <= 128:
        bwd_launches -= (1 if bags else 0) + 1

    def exchange_and_apply():
        if dist is not None:
            dist.all_reduce(dense, op=dist.ReduceOp.SUM)
        robe.robe_apply_sgd(h, dense, lr / world, True)  # mean of the ranks' gradients

    def step(i, events=None):
        k = i % NB
        if events is not None:
            events[0].record()
        if share_keys:
            robe.robe_forward_keep(h, d_ids[k], d_offs[k], B, out, ws)
        else:
            robe.robe_forward(h, d_ids[k], d_offs[k], B, out)
        if events is not None:
            events[1].record()
        if share_keys:
            robe.robe_backward_kept(h, grad_out, d_ids[k], d_offs[k], B, dense, lr, ws)
        else:
            robe.robe_backward(h, grad_out, d_ids[k], d_offs[k], B, dense, lr, ws)
        if events is not None:
            events[2].record()
        if dp_step:
            exchange_and_apply()
            if events is not None:
                events[3].record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(visible_gpu_index(local_rank))
    sampler.start()  # before the warm-up, so that samples are already coming when the timing starts
    for i in range(args.warmup):
        step(i)
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    t_start.record()
    for i in range(args.steps):
        step(args.warmup + i, evs[i])
    t_end.record()
    barrier()
    wall1 = time.time()
    clocks = sampler.stop((wall0, wall1))
    total_ms = t_start.elapsed_time(t_end)
    fwd_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    bwd_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    apply_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in evs])) if dp_step else 0.0
    if dp_step and not robe.dp.replicas_identical(array):
        raise RuntimeError("the replicas of the array differ after the data-parallel steps")
    nnz_per_step = float(np.mean([len(batches[(args.warmup + i) % NB][0]) for i in range(args.steps)]))

    # ---- end to end: host buffers in, result out, every step ------------------------------
    # Three streams, two sets of buffers: while step i computes, the inputs of step i+1 come in
    # from pinned host memory and the output of step i-1 goes back - what a caller that feeds the
    # library from the host would do.  Every byte of every step still crosses the bus inside
    # the timed region.
    # ids cross the bus as int32 when they fit (ROBE_OPT_INDEX_TYPE = ROBE_I32: half the id bytes)
    e2e_id_dtype = torch.int32 if max(int(b[0].max()) if len(b[0]) else 0 for b in batches) < 2**31 else id_dtype
    e2e_id_bytes = 4 if e2e_id_dtype == torch.int32 else 8
    h_ids = [torch.from_numpy(b[0]).to(e2e_id_dtype).pin_memory() for b in batches]
    h_offs = [None if b[1] is None else torch.from_numpy(b[1]).pin_memory() for b in batches]
    NBUF = args.e2e_buffers  # sets of device and pinned buffers the steps rotate through
    h_grad = grad_out.cpu().pin_memory()
    h_out = [torch.empty(B, T, d, dtype=torch.float32).pin_memory() for _ in range(NBUF)]
    max_nnz = max(len(b[0]) for b in batches)
    e_ids = [torch.empty(max_nnz, dtype=e2e_id_dtype, device=dev) for _ in range(NBUF)]
    e_offs = [torch.empty(nbags + 1, dtype=torch.int64, device=dev) if bags else None for _ in range(NBUF)]
    e_grad = [torch.empty_like(grad_out) for _ in range(NBUF)]
    e_out = [torch.empty_like(out) for _ in range(NBUF)]
    s_in, s_comp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(NBUF)]
    ev_comp = [torch.cuda.Event() for _ in range(NBUF)]
    ev_out = [torch.cuda.Event() for _ in range(NBUF)]

    def e2e_step(i):
        b, k = i % NBUF, i % NB
        n = h_ids[k].numel()
        ids_d = e_ids[b][:n]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_comp[b])  # the step that last read this set of inputs is done
            ids_d.copy_(h_ids[k], non_blocking=True)
            if bags:
                e_offs[b].copy_(h_offs[k], non_blocking=True)
            e_grad[b].copy_(h_grad, non_blocking=True)
            ev_in[b].record(s_in)
        s_comp.wait_event(ev_in[b])
        s_comp.wait_event(ev_out[b])     # the output buffer has been copied out
        if share_keys:
            robe.robe_forward_keep(h, ids_d, e_offs[b], B, e_out[b], ws, stream=s_comp)
            robe.robe_backward_kept(h, e_grad[b], ids_d, e_offs[b], B, dense, lr, ws, stream=s_comp)
        else:
            robe.robe_forward(h, ids_d, e_offs[b], B, e_out[b], stream=s_comp)
            robe.robe_backward(h, e_grad[b], ids_d, e_offs[b], B, dense, lr, ws, stream=s_comp)
        if dp_step:
            with torch.cuda.stream(s_comp):
                exchange_and_apply()
        ev_comp[b].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[b])
            h_out[b].copy_(e_out[b], non_blocking=True)
            ev_out[b].record(s_out)

    e2e_steps = max(4, min(args.steps, 20))
    for i in range(4):
        e2e_step(i)
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(s_in)
    for i in range(e2e_steps):
        e2e_step(i)
    s_out.wait_stream(s_comp)
    s_out.wait_stream(s_in)
    s1.record(s_out)
    barrier()
    e2e_ms = s0.elapsed_time(s1)
    e2e_nnz = float(np.mean([len(batches[i % NB][0]) for i in range(e2e_steps)]))
    h2d = int(e2e_id_bytes * e2e_nnz + (8 * (nbags + 1) if bags else 0) + 4 * nbags * d)
    d2h = int(4 * nbags * d)

    # ---- max over ranks --------------------------------------------------------------------
    (total_ms, e2e_ms, fwd_ms, bwd_ms, apply_ms), (job_ids, job_e2e_ids) = aggregate_over_ranks(
        dist, dev, [total_ms, e2e_ms, fwd_ms, bwd_ms, apply_ms],
        [nnz_per_step * args.steps, e2e_nnz * e2e_steps])

    robe.robe_destroy(h)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    peak, peak_kind = measured_peaks()
    fwd_bytes, bwd_bytes = algorithmic_bytes(w, nbags, nnz_per_step, bags, id_bytes)
    fwd_kernel = "fwd_staged_kernel" if d <= 128 else "fwd_direct_kernel"
    bwd_label = {"atomic": "bwd_atomic_staged_kernel" if d <= 128 else "bwd_atomic_direct_kernel",
                 "binned": "composite: keys, sort_count, sort_scan, sort_scatter, binned_apply kernels",
                 "det": "composite: keys, sort passes, window bounds/classes, apply kernels"}[args.backward]
    if share_keys:
        bwd_label = bwd_label.replace("keys, ", "")
    # a traffic record applies to the configuration it was captured on, and to no other
    own_batch = args.batch == 0
    rec = NCU_TRAFFIC_RECORDS.get((w.name, args.backward, bool(share_keys), args.ids, args.bag_layout)) \
        if (own_batch and not dp_step and world == 1 and args.fwd_kernel == 0 and args.bwd_kernel == 0
            and args.l2_keep == 0) else None
    sm_mhz = clocks.get("sm_mhz")

    def roof(nbytes, ms, kernel, which):
        ach = nbytes / (ms * 1e-3) / 1e9
        r = {"kernel": kernel, "bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s",
             "frac": ach / peak, "peak_kind": f"of {peak_kind}",
             "traffic": rec[which] if rec else None,
             "traffic_source": rec["source"] if rec else None,
             "ms_per_launch": ms, "algorithmic_bytes": int(nbytes)}
        if sm_mhz:
            r["ms_x_sm_mhz"] = ms * sm_mhz
        return r

    # The binned and the deterministic backward are built to keep the array's read-modify-write in
    # L2, so next to the survey's model (every add reads and writes its slot in HBM) they are also
    # read against the bytes such a path must move: ids, the block starts and payloads written and
    # read once per sort pass, one read and one write of the touched part of the array, and the
    # gradient elements once per id.
    touched = min(float(w.M), nnz_per_step * d) * 4
    npass_keys = {"atomic": 0, "binned": 1, "det": -(-max(1, (w.M - 1).bit_length()) // 8)}[args.backward]
    blocks = nnz_per_step * (-(-d // min(w.Z, d)))
    # per block: start and payload written once (8 B) and read by the apply (8 B); per sort pass
    # the starts read by the count (4 B), both read (8 B) and written (8 B) by the scatter
    key_bytes = blocks * (16 + 20 * npass_keys) if npass_keys else 0
    l2_rmw_bytes = (id_bytes * nnz_per_step + (8 * (nbags + 1) if bags else 0) + 2 * touched
                    + 4 * d * nnz_per_step + key_bytes)
    roof_b = roof(bwd_bytes, bwd_ms, bwd_label, "backward")
    roof_b["algorithmic_bytes_l2_rmw"] = int(l2_rmw_bytes)
    roof_b["frac_l2_rmw"] = l2_rmw_bytes / (bwd_ms * 1e-3) / 1e9 / peak

    value = job_ids / (total_ms * 1e-3)
    array_mb = w.M * (4 if w.array_dtype == "f32" else 2) / 1e6
    stream_mb = (2 * 4 * nbags * d + 8 * nnz_per_step) / 1e6
    if array_mb > 2 * 126:
        l2_note = f"{array_mb:.0f} MB array and 4 rotated id batches exceed L2; no flush"
    else:
        l2_note = (f"{array_mb:.0f} MB array stays L2-warm on purpose (steady state of a model that fits L2); "
                   f"the {stream_mb:.0f} MB of ids, output and gradient streamed per step exceed L2; no flush")
    if dp_step:
        parallelism = f"dp{world}, all-reduce of the dense gradient ({4 * w.M} bytes per rank and step), dense SGD apply"
    else:
        parallelism = f"dp{world}: one replica, fused SGD, nothing to exchange" if world == 1 else \
            f"dp{world} replicas, no collective"
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "num_tables": T, "d": d, "Z": w.Z, "M": w.M, "batch_per_gpu": B,
                   "ids_per_step_per_gpu": nnz_per_step, "ids": args.ids, "fwd_kernel": args.fwd_kernel, "l2_keep": l2_keep,
                   "bwd_kernel": args.bwd_kernel, "bags": bags, "bag_layout": args.bag_layout,
                   "backward": {"atomic": "atomic", "det": "deterministic", "binned": "binned atomic"}[args.backward] +
                   (", SGD fused" if dense is None else (", dense fp32 gradient, all-reduce, dense SGD apply" if dp_step
                                                         else ", dense fp32 gradient")),
                   "block_starts": ("hashed once per step: kept by the forward for the backward" if share_keys
                                    else "hashed by the forward and again by the backward"),
                   "l2": l2_note,
                   "parallelism": parallelism},
        "clocks": clocks,
        "e2e": {"value": job_e2e_ids / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "ids": "int32" if e2e_id_bytes == 4 else "int64",
                "ms_per_step": e2e_ms / e2e_steps},
        # forward kernel (+ the gap-fill kernel beside it when block starts of pooled input are kept),
        # the backward's kernels, the dense apply of the data-parallel step
        "gpu_launches": (1 + (1 if (share_keys and bags and d <= 128) else 0) + bwd_launches
                         + (1 if dp_step else 0)) * args.steps,
        # ONE kernel: the forward gather (the largest single kernel of the step by the ncu launch
        # list under profiles/, and the kernel the >= 0.60 target is stated for)
        "roofline": roof(fwd_bytes, fwd_ms, fwd_kernel, "forward"),
        "roofline_backward": roof_b,
        "forward_models": {k: {"bytes": int(v), "GB/s": v / (fwd_ms * 1e-3) / 1e9,
                               "frac": v / (fwd_ms * 1e-3) / 1e9 / peak}
                           for k, v in forward_byte_models(w, nbags, nnz_per_step, bags, id_bytes).items()},
        "forward_only": {"value": world * nnz_per_step / (fwd_ms * 1e-3), "unit": UNIT,
                         "bags_per_s": world * nbags / (fwd_ms * 1e-3), "ms": fwd_ms},
    }
    if dp_step:
        # all-reduce + apply together (the collective runs in the process group's own stream between
        # two events of the compute stream); the apply alone moves 12 bytes per slot
        line["exchange_and_apply"] = {"ms": apply_ms, "apply_algorithmic_bytes": 12 * w.M,
                                      "allreduce_bytes_per_rank": 4 * w.M}
    if not args.no_cpu_baseline and world == 1:
        sample_batch = w.batch  # about 10 s of host work on the default workload
        rate, n, threads, dt = oracle_step_rate(w, sample_batch, synth.array_to_numpy(array), variant=7)
        line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{sample_batch} of {w.batch} samples ({n} ids), forward "
                                          f"({threads} threads) + fp64 backward (1 thread), {dt:.1f} s"}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", help=WORKLOAD_HELP)
    ap.add_argument("--backward", default="auto", choices=["auto", "atomic", "binned", "det"],
                    help="backward variant of the step; auto = binned atomic adds when the array lives in "
                         "HBM and is touched several times per step, else plain atomic adds")
    ap.add_argument("--ids", default="int64", choices=["int64", "int32"], help="element type of the id arrays")
    ap.add_argument("--bag-layout", default="sample-major", choices=["sample-major", "table-major"],
                    help="bag numbering of the inputs: n*T + e (default) or e*B + n (per-table id lists end to end)")
    ap.add_argument("--fwd-kernel", type=int, default=0,
                    help="ROBE_OPT_FWD_KERNEL: 0 automatic, 1 direct, 2 staged (4-byte loads), 3 vector (16-byte loads)")
    ap.add_argument("--bwd-kernel", type=int, default=0,
                    help="ROBE_OPT_BWD_KERNEL of the atomic backward: 0 automatic, 1 direct, 2 staged, others see robe.h")
    ap.add_argument("--l2-keep", type=int, default=0, choices=[0, 1],
                    help="ROBE_OPT_ARRAY_L2_KEEP: 0 the backward's reductions carry the L2 evict-last policy "
                         "(default), 1 off")
    ap.add_argument("--e2e-buffers", type=int, default=2, choices=[2, 3, 4],
                    help="buffer sets of the end-to-end leg (copies of neighbouring steps overlap the compute)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dp-step", default="auto", choices=["auto", "on", "off"],
                    help="data-parallel step (backward into a dense gradient, all-reduce over the ranks, dense "
                         "SGD apply) instead of the fused SGD step; auto = on with more than one rank")
    ap.add_argument("--no-share-keys", dest="share_keys", action="store_false",
                    help="hash the ids in the backward again (robe_forward + robe_backward) instead of "
                         "keeping the forward's block starts (robe_forward_keep + robe_backward_kept)")
    ap.add_argument("--batch", type=int, default=0,
                    help="samples per GPU instead of the workload's own batch (small profiler captures)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    w = pick_workload(args.workload)
    if args.batch > 0:
        w = w.with_(batch=args.batch, name=f"{w.name}_batch{args.batch}")
    if args.impl == "reference":
        return run_reference(args, w)
    return run_ours(args, w)


if __name__ == "__main__":
    sys.exit(main())
