"""Benchmark of the TreeKV hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload cfg4] [--impl reference]

Headline (value): decode steps/s on the Llama-3-8B-shaped decode configuration (32 layers, batch 32, 32 query / 8 KV
heads, d=128, bf16, budget 2048) with every cache full, one step = all 32 layers in order, inputs resident in HBM.
A timed block is exactly K steps between two CUDA events; blocks are repeated back to back until the timed region
lasts at least a second, and the median block is reported (`blocks`, `region_ms` say how many and how long).
`e2e`: the same step through treekv_decode_step_host with page-locked host tensors: q, k, v cross the bus to the
GPU and the output crosses it back inside the timed region, every layer of every step (the kernel reads and writes
the host tensors itself; h2d / d2h bytes are counted from the tensors).
`decode_legs`: the same measurement on the other decode shapes (configuration 2; the decode phases of
configurations 5 and 3; configuration 1, which is launch-latency-bound), and the headline configuration once more with
in-cache positions (Section 4.1 "Position Encoding": keys rotated by cache slot inside the kernel).
`prefill` / `prefill_legs`: chunked-prefill tokens/s (through all layers), steady state with full chunks, on
configurations 5 (headline prefill), 4 and 3, each with a tensor roofline entry that gives the executed (three
contractions) and the two-contraction fractions against the sustained, burst and nominal bf16 peaks.
`roofline`: algorithmic bytes of one decode launch / its average duration, against the measured copy bandwidth.
`cpu_baseline`: the fp64 oracle timed on this host's cores on a bounded sample of the same workload (decode steps/s,
and prefill tokens/s under `prefill.cpu_baseline`).
`clocks`: nvidia-smi samples taken inside each leg's timed region (one sampler runs for the whole program).

With N > 1 (torchrun) every rank runs an independent replica of the workload (the path has no exchange step);
value is the sum over ranks, timed as the max over ranks.
"""
from __future__ import annotations

import argparse
import datetime
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
NOMINAL_HBM_GBS = 8000.0       # the figure the target is stated against
NOMINAL_BF16_TFLOPS = 2250.0   # dense bf16, nominal
MIN_REGION_MS = 1000.0         # a leg repeats its timed block until the region is at least this long


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                    "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


# ------------------------------------------------------------------------------------------------------
# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, valid for the named workload's per-layer shape and only while the kernel's sources are the ones that
# were profiled: a changed source file makes the entry stale and the reported traffic null.
NCU_TRAFFIC = {
    ('decode_mma_kernel', 'cfg4'): {"bytes_per_launch": 276873216, "sources": ['decode_mma.cu', 'common.cuh', 'tma.cuh'],
        "sha1": "7760273f6afd79fd142d87e0070cdb22723b8994", "profile": "profiles/decode_mma_cfg4_1layer.md"},
    ('decode_mma_kernel', 'cfg2'): {"bytes_per_launch": 140841472, "sources": ['decode_mma.cu', 'common.cuh', 'tma.cuh'],
        "sha1": "7760273f6afd79fd142d87e0070cdb22723b8994", "profile": "profiles/decode_mma_cfg2_1layer.md"},
    ('decode_mma_kernel', 'cfg5'): {"bytes_per_launch": 68887808, "sources": ['decode_mma.cu', 'common.cuh', 'tma.cuh'],
        "sha1": "7760273f6afd79fd142d87e0070cdb22723b8994", "profile": "profiles/decode_mma_cfg5_1layer.md"},
    ('decode_mma_kernel', 'cfg3'): {"bytes_per_launch": 33938944, "sources": ['decode_mma.cu', 'common.cuh', 'tma.cuh'],
        "sha1": "7760273f6afd79fd142d87e0070cdb22723b8994", "profile": "profiles/decode_mma_cfg3_1layer.md"},
    ('prefill_tc2_kernel', 'cfg5'): {"bytes_per_launch": 165460992, "sources": ['prefill_tc2.cu', 'prefill_tc_common.cuh', 'tma.cuh', 'common.cuh'],
        "sha1": "2005cb6e2d6cc6f07ec484540ac8d3c80dec117e", "profile": "profiles/prefill_tc2_cfg5_1layer.md"},
    ('prefill_tc2_kernel', 'cfg4'): {"bytes_per_launch": 1166141696, "sources": ['prefill_tc2.cu', 'prefill_tc_common.cuh', 'tma.cuh', 'common.cuh'],
        "sha1": "2005cb6e2d6cc6f07ec484540ac8d3c80dec117e", "profile": "profiles/prefill_tc2_cfg4_1layer.md"},
    ('prefill_tc_kernel', 'cfg3'): {"bytes_per_launch": 46809600, "sources": ['prefill_tc.cu', 'prefill_tc_common.cuh', 'tma.cuh', 'common.cuh'],
        "sha1": "c1b30800d0c447cec9ead6770a2a08397de9b4f1", "profile": "profiles/prefill_tc_cfg3_2layers.md"},
}


def measured_traffic(kernel, workload):
    import hashlib

    ent = NCU_TRAFFIC.get((kernel, workload))
    if ent is None:
        return None
    h = hashlib.sha1()
    try:
        for f in ent["sources"]:
            h.update(open(os.path.join(ROOT, "paper_2501_04987_b200", "csrc", f), "rb").read())
    except OSError:
        return None
    return ent["bytes_per_launch"] if h.hexdigest() == ent["sha1"] else None


# ------------------------------------------------------------------------------------------------------
# algorithmic bytes / flops
# ------------------------------------------------------------------------------------------------------
def decode_bytes_per_unit(c, d, e, g):
    """What one decode step must move per (sequence, KV head): K,V stream + S read/write + appended row + one
    survivor row read/write + q in, out."""
    return 2 * (c + 1) * d * e + 8 * (c + 1) + 2 * d * e + 4 * d * e + 2 * g * d * e


def prefill_flops_per_head_chunk(m, L, d, contractions=3):
    """Per query head and steady chunk; causal half of the diagonal block not counted.  contractions = 3: what the
    two-pass method executes (QK^T for the row statistics, QK^T again for the probabilities, PV); contractions = 2:
    what attention with column sums needs at the least (QK^T once, PV)."""
    return contractions * 2 * d * (m * L + m * (m + 1) // 2)


# ------------------------------------------------------------------------------------------------------
class ClockSampler:
    """One nvidia-smi sampler for the whole program; a leg asks for the samples that fell inside its timed region."""
    QUERY = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    BAD = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is not None:
            try:
                self.proc.terminate()
                self.proc.wait(timeout=5)
            except Exception:
                pass
            self.proc = None

    def cleanup(self):
        self.stop()
        try:
            if self.path:
                os.unlink(self.path)
        except OSError:
            pass

    def window(self, t0, t1):
        """Summary of the samples whose time stamp lies in [t0, t1] (host wall clock, seconds since the epoch)."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": [], "samples": 0}
        if self.path is None:
            return out
        sm, smmax, pw, reasons = [], [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 10:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    if ts < t0 or ts > t1:
                        continue
                    sm.append(float(f[2])); smmax.append(float(f[3]))
                    try:
                        pw.append(float(f[4]))
                    except ValueError:
                        pass
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[6:10]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        except OSError:
            return out
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smmax), reasons=sorted(reasons), samples=len(sm),
                       power_w=statistics.median(pw) if pw else None)
        return out

    @classmethod
    def rejected(cls, clocks):
        """A measurement taken under a hardware or thermal slowdown, or with the SM clock far below its maximum
        although nothing is throttling (a leftover clock lock), does not count."""
        if not clocks or not clocks.get("samples"):
            return False
        if any(r in cls.BAD for r in clocks["reasons"]):
            return True
        return not clocks["reasons"] and clocks["sm_mhz"] < 0.75 * clocks["sm_max_mhz"]


class Timer:
    """Timed blocks on the current CUDA stream: `run_block(i)` enqueues exactly the block's work; blocks are repeated
    back to back until the region lasts MIN_REGION_MS, each bracketed by CUDA events; the median block counts.
    The number of blocks is agreed over the ranks from a first, untimed block (one more warm-up)."""

    def __init__(self, torch, rep, sampler, min_region_ms=MIN_REGION_MS, max_blocks=5000):
        self.torch, self.rep, self.sampler = torch, rep, sampler
        self.min_region_ms, self.max_blocks = min_region_ms, max_blocks

    def measure(self, run_block):
        torch, rep = self.torch, self.rep
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        rep.barrier()
        e0.record(); run_block(-1); e1.record()
        rep.barrier()
        probe_ms = rep.max_over_ranks(e0.elapsed_time(e1))
        nblk = int(min(self.max_blocks, max(1, math.ceil(self.min_region_ms / max(probe_ms, 1e-3)))))
        for attempt in range(2):
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(nblk + 1)]
            rep.barrier()
            t0 = time.time()
            evs[0].record()
            for i in range(nblk):
                run_block(i)
                evs[i + 1].record()
            rep.barrier()
            t1 = time.time()
            blocks = [evs[i].elapsed_time(evs[i + 1]) for i in range(nblk)]
            clocks = self.sampler.window(t0, t1) if (self.sampler is not None and rep.rank == 0) else None
            if not ClockSampler.rejected(clocks):
                break
            if clocks is not None:
                clocks["remeasured_after"] = list(clocks["reasons"]) or ["sm clock far below max with no reason"]
        med = rep.max_over_ranks(statistics.median(blocks))
        return {"block_ms": med, "blocks": nblk, "region_ms": rep.max_over_ranks(evs[0].elapsed_time(evs[-1])),
                "block_ms_min": min(blocks), "block_ms_max": max(blocks), "clocks": clocks}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        ids = [x for x in vis.split(",") if x != ""]
        if local_rank < len(ids) and ids[local_rank].isdigit():
            return int(ids[local_rank])
    return local_rank


def whole_job_rate(world, units_per_rank, ms):
    """Units per second of all replicas together: every rank processed `units_per_rank` within `ms` (the max)."""
    return world * units_per_rank / (ms * 1e-3)


class Replicas:
    """The N > 1 plumbing: every rank runs an independent replica (the path has no exchange step), so the only
    collectives are the barrier around a timed region and the max of the ranks' device times.  `backend` "nccl"
    needs `device`; "gloo" runs the same logic on CPU ranks."""

    def __init__(self, backend="nccl", device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist

            if backend == "nccl":
                dist.init_process_group("nccl", device_id=device)
            else:
                dist.init_process_group(backend)
            self.dist = dist

    def barrier(self):
        """All ranks have reached this point and this rank's device is idle."""
        if self.dist is not None:
            self.dist.barrier()
        if self.device is not None:
            import torch

            torch.cuda.synchronize(self.device)

    def max_over_ranks(self, ms):
        if self.dist is None:
            return float(ms)
        import torch

        t = torch.tensor([ms], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank, ms):
        return whole_job_rate(self.world, units_per_rank, ms)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None


# ------------------------------------------------------------------------------------------------------
# oracle timing (cpu_baseline legs and --impl reference)
# ------------------------------------------------------------------------------------------------------
def _oracle_fill(orc, ws, upto):
    """Fill the oracle's caches to `upto` tokens with causal chunk passes of 256 tokens (not timed)."""
    t = 0
    while t < upto:
        n = min(256, upto - t)
        q, k, v = W.tokens(ws, 0, t, t + n)
        orc.prefill_chunk(q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3))
        t += n
    return t


def time_oracle_decode(w, seqs, steps):
    """Oracle decode steps/s for the whole configuration, from a sample of `seqs` sequences of one layer with
    full caches.  Returns (steps_per_s_full_config, cores, description)."""
    from oracle import Oracle

    ws = W.parity_slice(w, layers=1, batch=seqs)
    orc = Oracle(ws.budget, ws.n_heads, ws.n_kv_heads, ws.head_dim, ws.batch)
    t = _oracle_fill(orc, ws, ws.budget)
    q, k, v = W.tokens(ws, 0, t, t + steps)
    q, k, v = (np.ascontiguousarray(x, dtype=np.float64) for x in (q, k, v))
    t0 = time.perf_counter()
    for s in range(steps):
        orc.decode_step(q[s], k[s], v[s])
    dt = time.perf_counter() - t0
    layer_seq_steps_per_s = steps * seqs / dt
    full = layer_seq_steps_per_s / (w.layers * w.batch)
    cores = len(os.sched_getaffinity(0))
    desc = ("oracle decode on %d of %d sequences of 1 of %d layers, caches full, %d steps in %.1f s; scaled by "
            "(layers*batch)/(sample sequences) = %g" % (seqs, w.batch, w.layers, steps, dt, w.layers * w.batch / seqs))
    return full, cores, desc


def time_oracle_prefill(w, seqs, chunk_tokens):
    """Oracle chunked-prefill tokens/s (through all layers, whole batch) from one steady-state chunk of
    `chunk_tokens` tokens on `seqs` sequences of one layer with full caches."""
    from oracle import Oracle

    ws = W.parity_slice(w, layers=1, batch=seqs)
    orc = Oracle(ws.budget, ws.n_heads, ws.n_kv_heads, ws.head_dim, ws.batch)
    t = _oracle_fill(orc, ws, ws.budget)
    q, k, v = W.tokens(ws, 0, t, t + chunk_tokens)
    q, k, v = (np.ascontiguousarray(x.transpose(1, 0, 2, 3), dtype=np.float64) for x in (q, k, v))
    t0 = time.perf_counter()
    orc.prefill_chunk(q, k, v)
    dt = time.perf_counter() - t0
    # the whole configuration pushes batch * chunk tokens through `layers` layers; the sample did seqs * chunk in one
    tok_s = (seqs * chunk_tokens / dt) / w.layers
    cores = len(os.sched_getaffinity(0))
    desc = ("oracle prefill of one %d-token chunk into full caches (budget %d) on %d of %d sequences of 1 of %d layers in "
            "%.1f s; divided by the number of layers" % (chunk_tokens, w.budget, seqs, w.batch, w.layers, dt))
    return tok_s, cores, desc


def config_of(w, **extra):
    c = {"workload": w.name, "layers": w.layers, "batch_per_gpu": w.batch, "n_heads": w.n_heads, "n_kv_heads": w.n_kv_heads,
         "head_dim": w.head_dim, "budget": w.budget}
    c.update(extra)
    return c


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import build_oracle

    build_oracle()
    seqs = min(2, w.batch)
    steps = max(1, args.steps)
    # warm-up steps are part of the cache fill; each "step" of this arm is one oracle decode step of the sample
    val, cores, desc = time_oracle_decode(w, seqs, min(steps, 200))
    line = {
        "metric": "treekv_decode_steps_per_s", "value": val, "unit": "steps/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1000.0 / val, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
        "config": config_of(w, parallelism="oracle on the host cores of rank 0"),
        "cpu_baseline": {"value": val, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--decode-legs", default="cfg2,cfg5,cfg3,cfg1", help="other decode shapes to time ('' = none)")
    ap.add_argument("--prefill-legs", default="cfg5,cfg4,cfg3", help="prefill shapes to time, the first is `prefill` ('' = none)")
    ap.add_argument("--prefill-chunks", type=int, default=2, help="chunks per timed prefill block")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-eviction-stream", action="store_true",
                    help="prefill legs: keep every kernel of a chunk on the caller's stream (TREEKV_OPT_EVICTION_STREAM off)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-region-ms", type=float, default=MIN_REGION_MS)
    ap.add_argument("--prefill-path", type=int, default=0, help="TREEKV_OPT_PREFILL_PATH for the prefill legs; 0 = automatic")
    ap.add_argument("--prefill-key-split", type=int, default=0, help="TREEKV_OPT_PREFILL_KEY_SPLIT; 0 = automatic")
    ap.add_argument("--no-positions-leg", action="store_true",
                    help="skip the decode and prefill legs that repeat the first configuration with in-cache positions")
    ap.add_argument("--fill-by-image", action="store_true",
                    help="decode legs: fill the caches through treekv_import_state (one launch per layer) instead of "
                         "budget + 37 decode steps; for profiling runs")
    ap.add_argument("--decode-split", type=int, default=0, help="thread blocks per (sequence, KV head); 0 = automatic")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling small cases)")
    args = ap.parse_args()

    def cfg(name):
        w = W.CONFIGS[name]
        return W.parity_slice(w, layers=min(w.layers, args.layers)) if args.layers else w

    w = cfg(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rep = Replicas("nccl", dev)
    rank, world = rep.rank, rep.world

    from paper_2501_04987_b200 import _build

    if rank == 0:
        _build.build()
    rep.barrier()
    from paper_2501_04987_b200 import binding

    peaks = measured_peaks()
    sampler = None
    if rank == 0:
        sampler = ClockSampler(physical_gpu_index(local_rank))
        sampler.start()
    timer = Timer(torch, rep, sampler, args.min_region_ms)
    steps, warmup = max(1, args.steps), max(3, args.warmup)

    # ------------------------------------------------------------------ decode legs (the first is the headline, with e2e)
    dec = run_decode_leg(torch, binding, w, steps, warmup, not args.no_e2e, args.decode_split, dev, rep, timer, peaks,
                         args.fill_by_image)
    decode_legs = []
    for name in [x for x in args.decode_legs.split(",") if x and x != w.name]:
        decode_legs.append(run_decode_leg(torch, binding, cfg(name), steps, warmup, False, args.decode_split, dev, rep, timer,
                                          peaks, args.fill_by_image))

    if not args.no_positions_leg:
        decode_legs.append(run_decode_leg(torch, binding, w, steps, warmup, False, args.decode_split, dev, rep, timer, peaks,
                                          args.fill_by_image, positions=True))

    # ------------------------------------------------------------------ prefill legs
    prefill_legs = []
    for name in [x for x in args.prefill_legs.split(",") if x]:
        prefill_legs.append(run_prefill_leg(torch, binding, cfg(name), max(1, args.prefill_chunks), dev, rep, timer, peaks,
                                            not args.no_eviction_stream, args.prefill_path, args.prefill_key_split))
    prefill = prefill_legs[0] if prefill_legs else None
    if prefill_legs and not args.no_positions_leg:  # the first prefill configuration once more with in-cache positions
        prefill_legs.append(run_prefill_leg(torch, binding, cfg(prefill["config"]["workload"]), max(1, args.prefill_chunks), dev,
                                            rep, timer, peaks, not args.no_eviction_stream, args.prefill_path,
                                            args.prefill_key_split, positions=True))
    if sampler is not None:
        sampler.stop()

    # ------------------------------------------------------------------ oracle on the host cores
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        val, cores, desc = time_oracle_decode(w, min(2, w.batch), 400)
        cpu_baseline = {"value": val, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": desc}
        if prefill is not None:
            pw = cfg(prefill["config"]["workload"])
            pval, pcores, pdesc = time_oracle_prefill(pw, 1, pw.chunk)
            prefill["cpu_baseline"] = {"value": pval, "unit": "tokens/s", "cores": pcores, "kind": "oracle", "sample": pdesc}

    if rank == 0:
        bpl = dec["roofline"]["bytes_per_launch"]
        line = {
            "metric": "treekv_decode_steps_per_s", "value": dec["value"], "unit": "steps/s", "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": dec["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": config_of(w, parallelism="replicas x%d" % world,
                                l2="no flush: one step streams %.2f GB of K/V (%.0f MB per layer) through a 126 MB L2"
                                   % (w.layers * bpl / 1e9, bpl / 1e6)),
            "blocks": dec["blocks"], "region_ms": dec["region_ms"], "tokens_per_s": dec["value"] * w.batch,
            "e2e": dec["e2e"], "gpu_launches": dec["gpu_launches"], "clocks": dec["clocks"], "roofline": dec["roofline"],
            "cpu_baseline": cpu_baseline, "prefill": prefill, "decode_legs": decode_legs, "prefill_legs": prefill_legs[1:],
        }
        print(json.dumps(line))
    if sampler is not None:
        sampler.cleanup()
    rep.close()


def full_cache_image(torch, kv, w, n_seen, dev, seed):
    """A state image (layout of treekv_export_state) of full caches after n_seen > budget tokens: seeded Gaussian K / V
    with the recipe's outlier key channels, the newest `budget` stream positions, positive score sums."""
    units, c, d = w.batch * w.n_kv_heads, w.budget, w.head_dim
    e = 2 if w.dtype == "bf16" else 4
    tdtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    up = lambda x: (x + 255) // 256 * 256
    sizes = [units * c * d * e, units * c * d * e, units * c * 4, units * c * 4, w.batch * 4, w.batch * 4]
    offs = [0]
    for n in sizes:
        offs.append(offs[-1] + up(n))
    raw = torch.zeros(offs[-1] + 256, dtype=torch.uint8, device=dev)
    img = raw[(-raw.data_ptr()) % 256:][:offs[-1]]
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    K = torch.randn((units, c, d), device=dev, generator=g)
    K[..., W.outlier_channels(d, w.n_outliers)] *= 8.0
    V = torch.randn((units, c, d), device=dev, generator=g)
    pos = torch.arange(n_seen - c, n_seen, device=dev, dtype=torch.int32).repeat(units, 1)
    S = torch.rand((units, c), device=dev, generator=g) * (n_seen - pos).float()
    img[offs[0]:offs[0] + sizes[0]] = K.to(tdtype).contiguous().view(torch.uint8).reshape(-1)
    img[offs[1]:offs[1] + sizes[1]] = V.to(tdtype).contiguous().view(torch.uint8).reshape(-1)
    img[offs[2]:offs[2] + sizes[2]] = S.contiguous().view(torch.uint8).reshape(-1)
    img[offs[3]:offs[3] + sizes[3]] = pos.contiguous().view(torch.uint8).reshape(-1)
    img[offs[4]:offs[4] + sizes[4]] = torch.full((w.batch,), n_seen, dtype=torch.int32, device=dev).view(torch.uint8)
    return img


def run_decode_leg(torch, binding, w, steps, warmup, with_e2e, decode_split, dev, rep, timer, peaks, fill_by_image=False,
                   positions=False):
    """Decode steps/s of one configuration with every cache full; optionally the same through the host entry points."""
    e = 2 if w.dtype == "bf16" else 4
    tdtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    g = w.group
    world, rank = rep.world, rep.rank
    wr = W.parity_slice(w, seed=w.seed + 1000 * rank)
    ctxs = [binding.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, 0) for _ in range(w.layers)]
    if decode_split:
        for c in ctxs:
            c.set_option(binding.OPT_DECODE_SPLIT, decode_split)
    if positions:
        # in-cache positions (Section 4.1 "Position Encoding"): one cos / sin table by cache slot shared by every layer;
        # q and k then arrive unrotated (the same seeded values, taken as such: timing does not depend on them)
        cos, sin = (torch.from_numpy(x).to(dev) for x in W.rope_tables(w.budget + 1, w.head_dim, w.rope_base))
        for c in ctxs:
            c.set_positions(cos, sin)
    ring = 4
    ins = []
    for layer in range(w.layers):
        # every cache will be full and mid-cycle when timing starts; the ring holds positions near there
        q, k, v = W.tokens(wr, layer, w.budget + 37, w.budget + 37 + ring)
        ins.append(tuple(torch.from_numpy(x).to(dev).to(tdtype).contiguous() for x in (q, k, v)))
    outs = [torch.empty((w.batch, w.n_heads, w.head_dim), dtype=tdtype, device=dev) for _ in range(w.layers)]
    stream = torch.cuda.current_stream().cuda_stream
    handles = [c._h for c in ctxs]
    ptrs = [[(q[r].data_ptr(), k[r].data_ptr(), v[r].data_ptr()) for r in range(ring)] for (q, k, v) in ins]
    optrs = [o.data_ptr() for o in outs]
    step_fn = binding.lib.treekv_decode_step
    counter = [0]

    def decode_steps(n):
        for _ in range(n):
            r = counter[0] % ring
            counter[0] += 1
            for layer in range(w.layers):
                qp, kp, vp = ptrs[layer][r]
                st = step_fn(handles[layer], qp, kp, vp, optrs[layer], None, stream)
                if st != 0:
                    raise RuntimeError("treekv_decode_step: " + binding.status_string(st))

    if fill_by_image:
        # every cache full and 37 evictions into its cycle through the state image (one launch per layer) instead of
        # budget + 37 decode steps: for profiling runs, where every launch before the captured one costs time
        for layer, c in enumerate(ctxs):
            c.import_state(full_cache_image(torch, c, w, w.budget + 37, dev, wr.seed + layer), [w.budget + 37] * w.batch)
        for b in range(w.batch):
            assert ctxs[0].tokens_seen(b) == w.budget + 37
    else:
        decode_steps(w.budget + 37)   # fill every cache (untimed)
    decode_steps(warmup)          # warm-up
    launches0 = sum(c.stats()["kernel_launches"] for c in ctxs)
    t = timer.measure(lambda i: decode_steps(steps))
    launches = (sum(c.stats()["kernel_launches"] for c in ctxs) - launches0) // (t["blocks"] + 1)  # per timed block
    ms_per_step = t["block_ms"] / steps
    steps_per_s = whole_job_rate(world, steps, t["block_ms"])

    units = w.batch * w.n_kv_heads
    bytes_per_launch = units * decode_bytes_per_unit(w.budget, w.head_dim, e, g)
    launch_ms = ms_per_step / w.layers
    achieved = bytes_per_launch / (launch_ms * 1e-3) / 1e9
    kernel = "decode_mma_kernel" if w.dtype == "bf16" else "decode_kernel"
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": None if positions else measured_traffic(kernel, w.name),
                "peak_source": peaks["source"], "kernel": kernel, "bytes_per_launch": bytes_per_launch,
                "launch_us": launch_ms * 1e3, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}
    if bytes_per_launch < 20e6:
        roofline["note"] = ("launch-latency-bound: a launch moves %.1f MB, which the copy peak would stream in %.1f us"
                            % (bytes_per_launch / 1e6, bytes_per_launch / peaks["hbm_gbs"] / 1e3))

    e2e = None
    if with_e2e:
        # host buffers through the C ABI: pinned q,k,v copied in and the output copied back, every layer, every step
        nb_q = w.batch * w.n_heads * w.head_dim * e
        nb_k = w.batch * w.n_kv_heads * w.head_dim * e
        h_in = [tuple(x.cpu().pin_memory() for x in ins[layer]) for layer in range(w.layers)]
        h_out = [torch.empty((w.batch, w.n_heads, w.head_dim), dtype=tdtype).pin_memory() for _ in range(w.layers)]
        host_fn = binding.lib.treekv_decode_step_host
        hptrs = [[(q[r].data_ptr(), k[r].data_ptr(), v[r].data_ptr()) for r in range(ring)] for (q, k, v) in h_in]
        hoptrs = [o.data_ptr() for o in h_out]

        def e2e_steps(n):
            for _ in range(n):
                r = counter[0] % ring
                counter[0] += 1
                for layer in range(w.layers):
                    qp, kp, vp = hptrs[layer][r]
                    st = host_fn(handles[layer], qp, kp, vp, hoptrs[layer], None, stream)
                    if st != 0:
                        raise RuntimeError("treekv_decode_step_host: " + binding.status_string(st))

        e2e_steps(3)
        te = timer.measure(lambda i: e2e_steps(steps))
        e2e_ms = te["block_ms"] / steps
        e2e = {"value": whole_job_rate(world, steps, te["block_ms"]), "unit": "steps/s",
               "h2d_bytes_per_step": w.layers * (nb_q + 2 * nb_k), "d2h_bytes_per_step": w.layers * nb_q, "steps": steps,
               "ms_per_step": e2e_ms, "blocks": te["blocks"], "region_ms": te["region_ms"], "clocks": te["clocks"],
               "api": "treekv_decode_step_host, page-locked host q,k,v,out"}
    del ctxs, ins, outs
    torch.cuda.empty_cache()
    return {"metric": "treekv_decode_steps_per_s", "value": steps_per_s, "unit": "steps/s", "steps": steps,
            "ms_per_step": ms_per_step, "blocks": t["blocks"], "region_ms": t["region_ms"],
            "block_ms_min_max": [t["block_ms_min"], t["block_ms_max"]], "gpu_launches": int(launches),
            "clocks": t["clocks"], "roofline": roofline, "e2e": e2e, "tokens_per_s": steps_per_s * w.batch,
            "config": config_of(w, in_cache_positions=bool(positions))}


def run_prefill_leg(torch, binding, pw, n_chunks, dev, rep, timer, peaks, eviction_stream=True, prefill_path=0, key_split=0,
                    positions=False):
    tdtype = torch.bfloat16 if pw.dtype == "bf16" else torch.float32
    world, rank = rep.world, rep.rank
    m, c = pw.chunk, pw.budget
    ctxs = [binding.TreeKV(c, pw.n_heads, pw.n_kv_heads, pw.head_dim, pw.dtype, pw.batch, m) for _ in range(pw.layers)]
    if positions:  # in-cache positions (Section 4.1 "Position Encoding"): one table by cache slot for every layer
        cos, sin = (torch.from_numpy(x).to(dev) for x in W.rope_tables(c + m, pw.head_dim, pw.rope_base))
    for x in ctxs:
        if positions:
            x.set_positions(cos, sin)
        if eviction_stream:
            x.set_option(binding.OPT_EVICTION_STREAM, 1)
        if prefill_path:
            x.set_option(binding.OPT_PREFILL_PATH, prefill_path)
        if key_split:
            x.set_option(binding.OPT_PREFILL_KEY_SPLIT, key_split)
    wr = W.parity_slice(pw, seed=pw.seed + 1000 * rank)
    ins = []
    for layer in range(pw.layers):   # the same chunk values every call: timing does not depend on them
        q, k, v = W.tokens(wr, layer, c, c + m)
        ins.append(tuple(torch.from_numpy(np.ascontiguousarray(x.transpose(1, 0, 2, 3))).to(dev).to(tdtype) for x in (q, k, v)))
    out = torch.empty((pw.batch, m, pw.n_heads, pw.head_dim), dtype=tdtype, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    handles = [x._h for x in ctxs]
    ptrs = [(q.data_ptr(), k.data_ptr(), v.data_ptr()) for (q, k, v) in ins]
    optr = out.data_ptr()
    fn = binding.lib.treekv_prefill_chunk

    def run(n):
        for _ in range(n):
            for layer in range(pw.layers):
                qp, kp, vp = ptrs[layer]
                st = fn(handles[layer], qp, kp, vp, optr, None, m, stream)
                if st != 0:
                    raise RuntimeError("treekv_prefill_chunk: " + binding.status_string(st))

    run(c // m + 3)  # fill the caches, then three steady chunks as warm-up
    launches0 = sum(x.stats()["kernel_launches"] for x in ctxs)
    t = timer.measure(lambda i: run(n_chunks))
    launches = (sum(x.stats()["kernel_launches"] for x in ctxs) - launches0) // (t["blocks"] + 1)
    ms = t["block_ms"]
    tok_s = whole_job_rate(world, n_chunks * m * pw.batch, ms)
    # the library gives a thread block two 128-row query tiles once the one-tile grid covers the GPU at least twice
    tiles = pw.batch * pw.n_kv_heads * ((m * pw.group + 127) // 128)
    kernel = "prefill_tc2_kernel" if tiles >= 2 * torch.cuda.get_device_properties(dev).multi_processor_count else "prefill_tc_kernel"
    heads = pw.layers * pw.batch * pw.n_heads
    flops3 = heads * prefill_flops_per_head_chunk(m, c, pw.head_dim, 3)
    flops2 = heads * prefill_flops_per_head_chunk(m, c, pw.head_dim, 2)
    ach3 = flops3 * n_chunks / (ms * 1e-3) / 1e12
    ach2 = flops2 * n_chunks / (ms * 1e-3) / 1e12
    sus, burst = peaks["bf16_tflops_sustained"], peaks["bf16_tflops"]
    del ctxs, ins
    torch.cuda.empty_cache()
    return {"metric": "treekv_prefill_tokens_per_s", "value": tok_s, "unit": "tokens/s", "chunks_per_block": n_chunks,
            "blocks": t["blocks"], "region_ms": t["region_ms"], "ms_per_chunk_all_layers": ms / n_chunks,
            "gpu_launches": int(launches), "clocks": t["clocks"],
            "config": config_of(pw, chunk=m, eviction_stream=bool(eviction_stream), in_cache_positions=bool(positions),
                                l2="no flush: a chunk reads %.0f MB of K/V per layer and a layer is revisited %d layers later (126 MB L2)"
                                   % (2 * pw.batch * pw.n_kv_heads * (c + m) * pw.head_dim * 2 / 1e6, pw.layers)),
            "roofline": {"bound": "tensor", "achieved": ach3, "peak": sus, "unit": "TFLOP/s", "frac": ach3 / sus,
                         "counts": "executed flops: QK^T for the row statistics, QK^T again for the probabilities, PV",
                         "frac_of_burst": ach3 / burst, "frac_of_nominal_2250": ach3 / NOMINAL_BF16_TFLOPS,
                         "two_contractions": {"achieved": ach2, "frac": ach2 / sus, "frac_of_burst": ach2 / burst,
                                              "frac_of_nominal_2250": ach2 / NOMINAL_BF16_TFLOPS,
                                              "counts": "QK^T once and PV: what attention with column sums needs at the least"},
                         "traffic": None if positions else measured_traffic(kernel, pw.name), "kernel": kernel,
                         "peak_source": peaks["source"] + " (sustained; the timed region lasts a second or more)",
                         "flops_per_chunk_all_layers": flops3}}


if __name__ == "__main__":
    main()
