"""Benchmark of the TreeKV hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload cfg2] [--impl reference]

Headline (value): decode steps/s on the Llama-2-7B-shaped configuration (32 layers, batch 8, 32 heads, d=128,
bf16, budget 1024) with every cache full, one step = all 32 layers in order, inputs resident in HBM.
`e2e`: the same step through treekv_decode_step_host with page-locked host tensors: q, k, v cross the bus to the
GPU and the output crosses it back inside the timed region, every layer of every step (the kernel reads and writes
the host tensors itself; h2d / d2h bytes are counted from the tensors).
`prefill`: chunked-prefill tokens/s (through all layers) on the Llama-3-8B-shaped prefill configuration (batch 4,
chunks of 1024 to budget 4096), steady state with full chunks, with its own tensor roofline entry.
`decode_alt` / `prefill_alt`: the same two measurements on the other decode (Llama-3-8B GQA, batch 32, budget 2048)
and prefill (Llama-2-7B, chunks of 512 to budget 2048) configurations.
`roofline`: algorithmic bytes of one decode launch / its average duration, against the measured copy bandwidth.
`cpu_baseline`: the fp64 oracle timed on this host's cores on a bounded sample of the same workload.

With N > 1 (torchrun) every rank runs an independent replica of the workload (the path has no exchange step);
value is the sum over ranks, timed as the max over ranks.
"""
from __future__ import annotations

import argparse
import json
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
    "decode_mma_kernel": {"workload": "cfg2", "bytes_per_launch": 141.16e6, "sources": ["decode_mma.cu", "common.cuh"],
                          "sha1": "d588789f54b63eefdcc6510a26c23f77377158e2", "profile": "profiles/decode_mma_cfg2_2layers.md"},
    "prefill_tc2_kernel": {"workload": "cfg5", "bytes_per_launch": 149.87e6, "sources": ["prefill_tc2.cu", "tma.cuh", "common.cuh"],
                           "sha1": "b9140f2051a2ccaeac53170c2d4270cdd2053141", "profile": "profiles/prefill_tc2_cfg5_1layer.md"},
    "prefill_tc_kernel": {"workload": "cfg3", "bytes_per_launch": 46.60e6, "sources": ["prefill_tc.cu", "tma.cuh", "common.cuh"],
                          "sha1": "026cc9d2ef69ada63b6fe549d1ae7c7e09da95fd", "profile": "profiles/prefill_tc_cfg3_2layers.md"},
}


def measured_traffic(kernel, workload):
    import hashlib

    ent = NCU_TRAFFIC.get(kernel)
    if ent is None or ent["workload"] != workload:
        return None
    h = hashlib.sha1()
    try:
        for f in ent["sources"]:
            h.update(open(os.path.join(ROOT, "paper_2501_04987_b200", "csrc", f), "rb").read())
    except OSError:
        return None
    return ent["bytes_per_launch"] if h.hexdigest() == ent["sha1"] else None


# ------------------------------------------------------------------------------------------------------
# algorithmic bytes / flops (what the method must move or compute)
# ------------------------------------------------------------------------------------------------------
def decode_bytes_per_unit(c, d, e, g):
    """K,V stream + S read/write + appended row + one survivor row read/write + q in, out."""
    return 2 * (c + 1) * d * e + 8 * (c + 1) + 2 * d * e + 4 * d * e + 2 * g * d * e


def prefill_flops_per_head_chunk(m, L, d):
    """QK^T for the statistics, QK^T again for the probabilities, PV; causal half of the diagonal block not counted."""
    return 3 * 2 * d * (m * L + m * (m + 1) // 2)


# ------------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, smmax, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); smmax.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smmax), reasons=sorted(reasons), samples=len(sm))
        return out


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
# oracle timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------------
def time_oracle_decode(w, seqs, steps):
    """Oracle decode steps/s for the whole configuration, from a sample of `seqs` sequences of one layer with
    full caches.  Returns (steps_per_s_full_config, cores, description)."""
    from oracle import Oracle

    ws = W.parity_slice(w, layers=1, batch=seqs)
    orc = Oracle(ws.budget, ws.n_heads, ws.n_kv_heads, ws.head_dim, ws.batch)
    # fill the caches with one causal chunk pass per 256 tokens (not timed)
    t = 0
    while t < ws.budget:
        n = min(256, ws.budget - t)
        q, k, v = W.tokens(ws, 0, t, t + n)
        orc.prefill_chunk(q.transpose(1, 0, 2, 3), k.transpose(1, 0, 2, 3), v.transpose(1, 0, 2, 3))
        t += n
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


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import build_oracle

    build_oracle()
    seqs = min(2, w.batch)
    steps = max(1, args.steps)
    # warm-up steps are part of the cache fill; each "step" of this arm is one oracle decode step of the sample
    val, cores, desc = time_oracle_decode(w, seqs, min(steps, 400))
    line = {
        "metric": "treekv_decode_steps_per_s", "value": val, "unit": "steps/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1000.0 / val, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
        "config": {"workload": w.name, "layers": w.layers, "batch_per_gpu": w.batch, "n_heads": w.n_heads,
                   "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "budget": w.budget,
                   "parallelism": "oracle on the host cores of rank 0"},
        "cpu_baseline": {"value": val, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg4"])
    ap.add_argument("--prefill-workload", default="cfg5", choices=["cfg3", "cfg5"])
    ap.add_argument("--no-alt", action="store_true", help="skip the second decode and prefill configurations")
    ap.add_argument("--prefill-chunks", type=int, default=4, help="timed steady-state chunks (0 = skip the prefill leg)")
    ap.add_argument("--e2e-steps", type=int, default=64)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode-split", type=int, default=0, help="thread blocks per (sequence, KV head); 0 = automatic")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling small cases)")
    args = ap.parse_args()

    w = W.CONFIGS[args.workload]
    if args.layers:
        w = W.parity_slice(w, layers=args.layers)
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
    barrier, max_over_ranks = rep.barrier, rep.max_over_ranks

    # ------------------------------------------------------------------ decode leg (headline) + e2e
    dec = run_decode_leg(torch, binding, w, args.steps, max(3, args.warmup), args.e2e_steps, args.decode_split, dev, world,
                         rank, local_rank, barrier, max_over_ranks, peaks, sample_clocks=True)
    steps_per_s, ms_per_step, launches = dec["value"], dec["ms_per_step"], dec["gpu_launches"]
    roofline, e2e, clocks, bytes_per_launch = dec["roofline"], dec["e2e"], dec["clocks"], dec["roofline"]["bytes_per_launch"]
    decode_alt = None
    if not args.no_alt:
        wa = W.CONFIGS["cfg4" if w.name == "cfg2" else "cfg2"]
        if args.layers:
            wa = W.parity_slice(wa, layers=args.layers)
        decode_alt = run_decode_leg(torch, binding, wa, max(16, args.steps // 4), 3, 0, args.decode_split, dev, world, rank,
                                    local_rank, barrier, max_over_ranks, peaks, sample_clocks=False)

    # ------------------------------------------------------------------ prefill leg
    prefill = None
    if args.prefill_chunks > 0:
        pw = W.CONFIGS[args.prefill_workload]
        if args.layers:
            pw = W.parity_slice(pw, layers=args.layers)
        prefill = run_prefill_leg(torch, binding, pw, args.prefill_chunks, dev, world, rank, barrier, max_over_ranks, peaks)
    prefill_alt = None
    if args.prefill_chunks > 0 and not args.no_alt:
        pa = W.CONFIGS["cfg3" if args.prefill_workload == "cfg5" else "cfg5"]
        if args.layers:
            pa = W.parity_slice(pa, layers=args.layers)
        prefill_alt = run_prefill_leg(torch, binding, pa, args.prefill_chunks, dev, world, rank, barrier, max_over_ranks, peaks)

    # ------------------------------------------------------------------ oracle on the host cores
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        val, cores, desc = time_oracle_decode(w, min(2, w.batch), 300)
        cpu_baseline = {"value": val, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {
            "metric": "treekv_decode_steps_per_s", "value": steps_per_s, "unit": "steps/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "layers": w.layers, "batch_per_gpu": w.batch, "n_heads": w.n_heads,
                       "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "budget": w.budget,
                       "parallelism": "replicas x%d" % world,
                       "l2": "no flush: one step streams %.2f GB of K/V (%.0f MB per layer) through a 126 MB L2"
                             % (w.layers * bytes_per_launch / 1e9, bytes_per_launch / 1e6)},
            "tokens_per_s": steps_per_s * w.batch,
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline,
            "cpu_baseline": cpu_baseline, "prefill": prefill, "decode_alt": decode_alt, "prefill_alt": prefill_alt,
        }
        print(json.dumps(line))
    rep.close()


def run_decode_leg(torch, binding, w, steps, warmup, e2e_steps, decode_split, dev, world, rank, local_rank, barrier,
                   max_over_ranks, peaks, sample_clocks):
    """Decode steps/s of one configuration with every cache full; optionally the same through the host entry points."""
    e = 2 if w.dtype == "bf16" else 4
    tdtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    g = w.group
    wr = W.parity_slice(w, seed=w.seed + 1000 * rank)
    ctxs = [binding.TreeKV(w.budget, w.n_heads, w.n_kv_heads, w.head_dim, w.dtype, w.batch, 0) for _ in range(w.layers)]
    if decode_split:
        for c in ctxs:
            c.set_option(binding.OPT_DECODE_SPLIT, decode_split)
    ring = 4
    ins = []
    for layer in range(w.layers):
        # every cache will be full and mid-cycle when timing starts; the ring holds positions near there
        q, k, v = W.tokens(wr, layer, w.budget + 37, w.budget + 37 + ring)
        ins.append(tuple(torch.from_numpy(x).to(dev).to(tdtype).contiguous() for x in (q, k, v)))
    outs = [torch.empty((w.batch, w.n_heads, w.head_dim), dtype=tdtype, device=dev) for _ in range(w.layers)]
    stream = torch.cuda.current_stream().cuda_stream

    def decode_steps(n, start):
        for s in range(start, start + n):
            r = s % ring
            for layer in range(w.layers):
                q, k, v = ins[layer]
                st = binding.lib.treekv_decode_step(ctxs[layer]._h, q[r].data_ptr(), k[r].data_ptr(), v[r].data_ptr(),
                                                    outs[layer].data_ptr(), None, stream)
                if st != 0:
                    raise RuntimeError("treekv_decode_step: " + binding.status_string(st))

    fill = w.budget + 37
    decode_steps(fill, 0)          # fill every cache (untimed)
    decode_steps(warmup, fill)     # warm-up
    launches0 = sum(c.stats()["kernel_launches"] for c in ctxs)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    barrier()
    if rank == 0 and sample_clocks:
        sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    decode_steps(steps, fill + warmup)
    ev1.record()
    barrier()
    clocks = sampler.stop() if (rank == 0 and sample_clocks) else None
    ms_total = max_over_ranks(ev0.elapsed_time(ev1))
    launches = sum(c.stats()["kernel_launches"] for c in ctxs) - launches0
    ms_per_step = ms_total / steps
    steps_per_s = whole_job_rate(world, steps, ms_total)

    units = w.batch * w.n_kv_heads
    bytes_per_launch = units * decode_bytes_per_unit(w.budget, w.head_dim, e, g)
    launch_ms = ms_total / (steps * w.layers)
    achieved = bytes_per_launch / (launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"],
                "traffic": measured_traffic("decode_mma_kernel" if w.dtype == "bf16" else "decode_kernel", w.name),
                "peak_source": peaks["source"],
                "kernel": "decode_mma_kernel" if w.dtype == "bf16" else "decode_kernel",
                "bytes_per_launch": bytes_per_launch, "launch_us": launch_ms * 1e3, "frac_of_nominal_8TBs": achieved / 8000.0}

    e2e = None
    if e2e_steps > 0:
        # host buffers through the C ABI: pinned q,k,v copied in and the output copied back, every layer, every step
        nb_q = w.batch * w.n_heads * w.head_dim * e
        nb_k = w.batch * w.n_kv_heads * w.head_dim * e
        h_in = [tuple(x.cpu().pin_memory() for x in ins[layer]) for layer in range(w.layers)]
        h_out = [torch.empty((w.batch, w.n_heads, w.head_dim), dtype=tdtype).pin_memory() for _ in range(w.layers)]

        def e2e_run(n):
            for s in range(n):
                r = s % ring
                for layer in range(w.layers):
                    q, k, v = h_in[layer]
                    st = binding.lib.treekv_decode_step_host(ctxs[layer]._h, q[r].data_ptr(), k[r].data_ptr(),
                                                             v[r].data_ptr(), h_out[layer].data_ptr(), None, stream)
                    if st != 0:
                        raise RuntimeError("treekv_decode_step_host: " + binding.status_string(st))

        e2e_n = max(1, min(e2e_steps, steps))
        e2e_run(3)
        barrier()
        ev0.record()
        e2e_run(e2e_n)
        ev1.record()
        barrier()
        e2e_ms = max_over_ranks(ev0.elapsed_time(ev1)) / e2e_n
        e2e = {"value": whole_job_rate(world, 1, e2e_ms), "unit": "steps/s", "h2d_bytes_per_step": w.layers * (nb_q + 2 * nb_k),
               "d2h_bytes_per_step": w.layers * nb_q, "steps": e2e_n, "ms_per_step": e2e_ms}
    del ctxs, ins, outs
    torch.cuda.empty_cache()
    return {"metric": "treekv_decode_steps_per_s", "value": steps_per_s, "unit": "steps/s", "steps": steps,
            "ms_per_step": ms_per_step, "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "e2e": e2e,
            "tokens_per_s": steps_per_s * w.batch,
            "config": {"workload": w.name, "layers": w.layers, "batch_per_gpu": w.batch, "n_heads": w.n_heads,
                       "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "budget": w.budget}}


def run_prefill_leg(torch, binding, pw, n_chunks, dev, world, rank, barrier, max_over_ranks, peaks):
    tdtype = torch.bfloat16 if pw.dtype == "bf16" else torch.float32
    m, c = pw.chunk, pw.budget
    ctxs = [binding.TreeKV(c, pw.n_heads, pw.n_kv_heads, pw.head_dim, pw.dtype, pw.batch, m) for _ in range(pw.layers)]
    wr = W.parity_slice(pw, seed=pw.seed + 1000 * rank)
    ring = 1  # the same chunk values every call: timing does not depend on them
    ins = []
    for layer in range(pw.layers):
        chunks = []
        for r in range(ring):
            q, k, v = W.tokens(wr, layer, c + r * m, c + (r + 1) * m)
            chunks.append(tuple(torch.from_numpy(np.ascontiguousarray(x.transpose(1, 0, 2, 3))).to(dev).to(tdtype)
                                for x in (q, k, v)))
        ins.append(chunks)
    out = torch.empty((pw.batch, m, pw.n_heads, pw.head_dim), dtype=tdtype, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def run(n, start):
        for s in range(start, start + n):
            for layer in range(pw.layers):
                q, k, v = ins[layer][s % ring]
                st = binding.lib.treekv_prefill_chunk(ctxs[layer]._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                                      out.data_ptr(), None, m, stream)
                if st != 0:
                    raise RuntimeError("treekv_prefill_chunk: " + binding.status_string(st))

    fill_chunks = c // m
    run(fill_chunks + 3, 0)  # fill the caches, then three steady chunks as warm-up
    launches0 = sum(x.stats()["kernel_launches"] for x in ctxs)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    run(n_chunks, fill_chunks + 3)
    ev1.record()
    barrier()
    ms = max_over_ranks(ev0.elapsed_time(ev1))
    launches = sum(x.stats()["kernel_launches"] for x in ctxs) - launches0
    tok_s = whole_job_rate(world, n_chunks * m * pw.batch, ms)
    # the library gives a thread block two 128-row query tiles once the one-tile grid covers the GPU at least twice
    tiles = pw.batch * pw.n_kv_heads * ((m * pw.group + 127) // 128)
    kernel = "prefill_tc2_kernel" if tiles >= 2 * torch.cuda.get_device_properties(dev).multi_processor_count else "prefill_tc_kernel"
    flops_chunk = pw.layers * pw.batch * pw.n_heads * prefill_flops_per_head_chunk(m, c, pw.head_dim)
    achieved = flops_chunk * n_chunks / (ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    del ctxs, ins
    torch.cuda.empty_cache()
    return {"metric": "treekv_prefill_tokens_per_s", "value": tok_s, "unit": "tokens/s", "chunks": n_chunks,
            "ms_per_chunk_all_layers": ms / n_chunks, "gpu_launches": int(launches),
            "config": {"workload": pw.name, "layers": pw.layers, "batch_per_gpu": pw.batch, "n_heads": pw.n_heads,
                       "n_kv_heads": pw.n_kv_heads, "head_dim": pw.head_dim, "budget": c, "chunk": m,
                       "l2": "no flush: a chunk reads %.0f MB of K/V per layer and a layer is revisited %d layers later (126 MB L2)"
                             % (2 * pw.batch * pw.n_kv_heads * (c + m) * pw.head_dim * 2 / 1e6, pw.layers)},
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                         "frac": achieved / peak, "traffic": measured_traffic(kernel, pw.name),
                         "kernel": kernel, "peak_source": peaks["source"] + " (sustained)",
                         "flops_per_chunk_all_layers": flops_chunk}}


if __name__ == "__main__":
    main()
