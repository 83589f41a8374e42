#!/usr/bin/env python
"""FO-SGD round-trip benchmark: gradient elements/s through encode -> server aggregate (+ downlink
encode) -> downlink decode, M simulated workers per GPU, synthetic gradients.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 0..4] [--block-log2 b] [--impl reference]

Prints ONE JSON line (rank 0).  With --gpus N > 1 and no launcher environment it starts the N ranks
itself.  `--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "FO-SGD round-trip gradient elems/s"
UNIT = "elems/s"
NOMINAL_HBM_GBS = 8000.0
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="index into the five workloads")
    ap.add_argument("--block-log2", type=int, default=0, help="0 = one global transform (the paper's scheme)")
    ap.add_argument("--impl", default="fosgd", choices=["fosgd", "reference"])
    ap.add_argument("--ws-workers", type=int, default=0, help="workers per launch the scratch buffer holds (0 = all)")
    ap.add_argument("--workers", type=int, default=0, help="override the workload's worker count (profiling of small cases)")
    ap.add_argument("--resident", type=int, default=0,
                    help="gradient rows kept on the device; fewer than the worker count streams the workers in "
                         "chunks of this many rows into one accumulator (default: all, 8 for the 1.3B workload)")
    ap.add_argument("--device-amplitudes", choices=["global", "block"], default=None,
                    help="measure the amplitudes on the device every step (one more read of the gradients) instead "
                         "of passing precomputed ones: one for all workers, or one per worker and block")
    ap.add_argument("--encode-streams", type=int, default=1,
                    help="run the uplink encoder's workers as this many sub-batches on side streams")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="repeat the block of --steps timed steps until this much device time has been timed")
    ap.add_argument("--fused-encoder", action="store_true",
                    help="run the uplink encoder of a 2^24-long transform as one kernel instead of two")
    ap.add_argument("--tensor-core-pass", type=int, default=None, choices=[0, 1, 2, 3],
                    help="decoder passes on the tensor cores: 1 = strided, 2 = contiguous, 3 = both (default: the library's)")
    ap.add_argument("--ws-factor", type=float, default=1.0,
                    help="scratch as a multiple of the minimum per worker (1.5: a decoder with two strided passes keeps its first pass in fp16)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the extra workloads, the K > 1 downlink table and the issue-rate probe")
    ap.add_argument("--e2e-pieces", type=int, default=16,
                    help="end-to-end leg: pieces the host-to-device copy is cut into (compute overlaps the later ones)")
    return ap.parse_args()


def kernel_source_digest():
    """Short hash of the kernel sources: ncu traffic figures are only quoted for the sources they came from."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2405_11095_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()[:12]


def measured_traffic(label, units):
    """DRAM bytes per launch of kernel `label` from profiles/dram_traffic.txt (ncu dram__bytes_read.sum +
    dram__bytes_write.sum per worker-coordinate, captured on a smaller case), or None if the file has no
    entry for this kernel or was taken from other kernel sources."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    family = label.split("@")[0]
    digest = kernel_source_digest()
    with open(path) as f:
        for line in f:
            parts = line.split()
            if len(parts) >= 3 and not line.startswith("#") and parts[0] == family and parts[2] == digest:
                return float(parts[1]) * units
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    def __init__(self, gpu_index: int):
        self.path = f"/tmp/fosgd_clocks_{os.getpid()}_{time.monotonic_ns()}.csv"
        self.proc = None
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={CLOCK_QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(gpu_index)], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.out.close()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    smax.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- CPU oracle timing
def oracle_sample(w, block_log2, steps, warmup):
    """Time the oracle's round trip on a bounded sample: m = min(cores, M) workers at full length,
    run side by side on the host cores (the oracle itself is serial), plus one downlink
    encode + decode.  Work is linear in the number of workers, so the time for all M workers
    is (M/m) * t_workers + t_downlink."""
    import numpy as np

    import oracle
    from paper_2405_11095_b200 import synthetic
    from concurrent.futures import ThreadPoolExecutor

    cores = os.cpu_count() or 1
    m = max(1, min(cores, w.M))
    d = w.d
    g = synthetic.gradients(w, "cpu", range(m)).double().numpy()
    dp = oracle.padded_dim(d, block_log2)
    n_eff = oracle.transform_len(d, block_log2)
    lam = oracle.lam(float(np.linalg.norm(g, axis=1).max()), w.alpha, n_eff)
    lam_s = oracle.lam_server(lam, w.alpha_s, n_eff)
    seed = 0

    def one_worker(n, step):
        bits = oracle.encode(g[n], seed, step, n, lam, block_log2=block_log2)
        return oracle.decode_full(bits, d, seed, step, n, lam, block_log2=block_log2)

    t_begin = time.perf_counter()
    t0 = time.perf_counter()
    gbar = np.mean([one_worker(0, 0)], axis=0)
    pl = oracle.downlink_encode(gbar, seed, 0, lam_s, K=w.K, block_log2=block_log2)
    oracle.downlink_decode(pl, dp, seed, 0, lam_s, K=w.K, block_log2=block_log2)
    t_first = time.perf_counter() - t0
    t0 = time.perf_counter()
    pl = oracle.downlink_encode(gbar, seed, 1, lam_s, K=w.K, block_log2=block_log2)
    oracle.downlink_decode(pl, dp, seed, 1, lam_s, K=w.K, block_log2=block_log2)
    t_down = time.perf_counter() - t0

    times = []
    with ThreadPoolExecutor(max_workers=m) as ex:
        for s in range(warmup + steps):
            t0 = time.perf_counter()
            list(ex.map(lambda n: one_worker(n, s), range(m)))
            if s >= warmup:
                times.append(time.perf_counter() - t0)
    t_workers = sum(times) / len(times)
    t_all = (w.M / m) * t_workers + t_down
    return {"value": w.M * d / t_all, "unit": UNIT, "cores": m, "kind": "oracle",
            "sample": f"{m} of {w.M} workers encoded+decoded at full d={d} on {m} threads "
                      f"({t_workers:.2f} s), one downlink encode+decode ({t_down:.2f} s), "
                      f"extrapolated linearly in M; first call {t_first:.2f} s untimed",
            "seconds_per_step_all_workers": t_all,
            "seconds_timed_per_step": t_workers + t_down,
            "seconds_wall_total": time.perf_counter() - t_begin}


def resident_rows(args, w):
    return args.resident or (8 if w.d > (1 << 30) else w.M)


def workload_config(w, args, world):
    R = resident_rows(args, w)
    return {"workload": w.name, "d": w.d, "workers_per_gpu": w.M, "workers_total": w.M * world,
            "input_dtype": str(w.dtype).replace("torch.", ""), "K_downlink": w.K,
            "block_log2": args.block_log2, "alpha": w.alpha, "alpha_s": w.alpha_s,
            "encode_streams": args.encode_streams,
            "amplitudes": f"measured on the device every step ({args.device_amplitudes})" if args.device_amplitudes
                          else "passed by value",
            "l2": "inputs exceed L2" if w.M * w.d * (2 if "bfloat16" in str(w.dtype) else 4) > 126e6 * 2
                  else "L2 flushed between steps",
            "parallelism": f"workers sharded over {world} GPU(s); one fp32 all-reduce of the partial average"
                           if world > 1 else "single GPU",
            "resident_gradient_rows": R, "streamed_chunks": w.M // R}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2405_11095_b200 import synthetic
    w = synthetic.WORKLOADS[args.config]
    if args.workers:
        w = dataclasses.replace(w, M=args.workers, name=f"{w.name}_workers{args.workers}")
    # bound the run: a timed step is one m-worker uplink sample (seconds), so cap the count
    steps = max(1, min(args.steps, 5))
    warmup = max(0, min(args.warmup, 1))
    r = oracle_sample(w, args.block_log2, steps, warmup)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    line = {"impl": "reference", "device": "cpu", "metric": METRIC, "value": r["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": steps, "warmup": warmup,
            "ms_per_step": 1e3 * r["seconds_per_step_all_workers"],
            "ms_per_step_is": "linear extrapolation in the worker count from the timed sample",
            "seconds_timed_per_step": r["seconds_timed_per_step"], "seconds_wall_total": r["seconds_wall_total"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args, 1 if world < 1 else 1),
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- byte and operation counts
def label_parts(label):
    name, workers = label.split("@")
    src, sink = name.split(":")[1].split("->")
    return src, sink, 1 if workers == "srv" else int(workers)


def implementation_bytes(label, dp, P):
    """Bytes one launch moves as implemented: its own source and sink, intermediates included."""
    src, sink, workers = label_parts(label)
    per = {"f32": 4.0, "bf16": 2.0, "bits": P / 8.0, "ws": 4.0, "ws16": 2.0}[src]
    per += {"ws": 4.0, "ws16": 2.0, "pack1": 1 / 8.0, "packK": P / 8.0, "final": 0.0, "amp": 0.0}[sink]
    if label.startswith("fused"):
        per += 8.0   # both passes in one kernel: the fp32 intermediate is written and read inside it
    return per * workers * dp + (4.0 * dp if sink == "final" else 0.0)


def algorithmic_bytes(label, d, dp, P):
    """The share of the method's own traffic that this launch carries: gradients in (true length d),
    packed words in or out, the accumulator or decoded vector out once per launch.  Intermediates
    between the passes of one transform are the implementation's, not the method's: zero here."""
    src, sink, workers = label_parts(label)
    b = {"f32": 4.0 * d, "bf16": 2.0 * d, "bits": P / 8.0 * dp, "ws": 0.0, "ws16": 0.0}[src] * workers
    b += {"ws": 0.0, "ws16": 0.0, "pack1": dp / 8.0 * workers, "packK": P * dp / 8.0 * workers, "final": 4.0 * dp,
          "amp": 0.0}[sink]
    return b


def is_uplink_kernel(k):
    # ("col..:ws->ws" is an encoder's middle pass, "dcol..:ws->ws" a decoder's)
    return "f32->" in k or "bf16->" in k or "->pack" in k or (k.startswith("col") and "ws->ws" in k)


# --------------------------------------------------------------------------- one workload on the GPU
def run_workload(env, args, w, steps, warmup, min_seconds, want_e2e):
    """Time the round trip of workload `w`; returns the record (all ranks compute it, rank 0 uses it)."""
    import torch
    import torch.distributed as dist

    F, D, synthetic = env["F"], env["D"], env["synthetic"]
    dev, rank, world, local_rank = env["dev"], env["rank"], env["world"], env["local_rank"]
    b = args.block_log2
    d, M = w.d, w.M
    dp = F.padded_dim(d, b)
    n_eff = F.transform_len(d, b)
    P = F.planes(w.K)
    esize = 2 if w.dtype == torch.bfloat16 else 4
    stride = (d + 7) // 8 * 8

    # inputs (untimed): this rank's workers, or the resident rows that the streamed workers cycle through
    R = resident_rows(args, w)
    if M % R:
        raise SystemExit("--resident must divide the worker count")
    grads = torch.zeros(R, stride, dtype=w.dtype, device=dev)
    for n in range(R):
        synthetic.worker_gradient(w, rank * M + n, dev, out=grads[n, :d])
    B = synthetic.norm_bound(grads[:, :d])
    if world > 1:
        t = torch.tensor([B], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        B = float(t.item())
    lam = F.lambda_(B, w.alpha, n_eff)
    lam_s = F.lambda_server(lam, w.alpha_s, n_eff)

    ws_per = F.workspace_bytes(F.OP_AGGREGATE, d, block_log2=b, K=w.K)
    ws_workers = args.ws_workers or R
    # (+ the progress words with which the one-kernel encoder takes all its workers in one launch)
    ws = torch.empty(max(16, int(ws_per * ws_workers * args.ws_factor) // 16 * 16 + F.fused_sync_bytes(ws_workers)), dtype=torch.uint8, device=dev) if ws_per else None
    buf = D.RoundTripBuffers(bits=torch.zeros(R, dp // 32, dtype=torch.int32, device=dev),
                             acc=torch.zeros(dp, dtype=torch.float32, device=dev),
                             down=torch.zeros(P, dp // 32, dtype=torch.int32, device=dev),
                             out=torch.zeros(d, dtype=torch.float32, device=dev), ws=ws)
    flush = None
    if R * d * esize <= 2 * 126e6:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    amps = None
    if args.device_amplitudes:
        pb = args.device_amplitudes == "block"
        if pb and not b:
            raise SystemExit("--device-amplitudes block needs --block-log2")
        nb = dp >> b if pb else 1
        amps = D.DeviceAmplitudes(
            lam=torch.zeros(R * nb if pb else 1, dtype=torch.float32, device=dev),
            lam_s=torch.zeros(nb, dtype=torch.float32, device=dev),
            ws=torch.empty(F.workspace_bytes(F.OP_BLOCK_AMPLITUDES if pb else F.OP_AMPLITUDES, d, M=R, block_log2=b),
                           dtype=torch.uint8, device=dev),
            per_block=pb, alpha=w.alpha, alpha_s=w.alpha_s)

    def step(s):
        return D.round_trip(F, grads, d, buf, lam, lam_s, 0, s, K=w.K, block_log2=b, rank=rank, world=world,
                            worker_stride=stride, workers=M, amps=amps,
                            encode_streams=args.encode_streams)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for s in range(warmup):
        step(s)
    barrier()

    # ---- timed region: blocks of K steps, each bracketed by barrier + synchronize; device time from
    # CUDA events around every step, per-kernel events through the library's trace hook.  Blocks
    # repeat until min_seconds of device time have been timed; the median block is reported. ----
    K = steps
    traces = [F.PassTrace(256) for _ in range(K)]
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    sampler = ClockSampler(local_rank) if rank == 0 else None
    block_ms, per, order, nblocks, timed_ms = [], {}, [], 0, 0.0
    while True:
        barrier()
        for s in range(K):
            if flush is not None:
                flush.fill_(s & 0xFF)
            ev[s][0].record()
            with traces[s]:
                step(1000 + nblocks * K + s)
            ev[s][1].record()
        barrier()
        total_ms = torch.tensor([sum(a.elapsed_time(bb) for a, bb in ev)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
        block_ms.append(float(total_ms.item()))
        timed_ms += block_ms[-1]
        nblocks += 1
        for tr in traces:
            for lab, ms in tr.durations_ms():
                if lab not in per:
                    per[lab] = [0.0, 0]
                    order.append(lab)
                per[lab][0] += ms
                per[lab][1] += 1
        if timed_ms >= 1e3 * min_seconds or nblocks >= 500:
            break
    clocks = sampler.stop() if sampler else None
    ms_per_step = statistics.median(block_ms) / K
    value = (M * world) * d / (ms_per_step * 1e-3)
    nsteps = K * nblocks
    kernels = {lab: {"launches_per_step": per[lab][1] / nsteps, "ms_per_launch": per[lab][0] / per[lab][1],
                     "ms_per_step": per[lab][0] / nsteps} for lab in order}
    launches_per_step = sum(c for _, c in per.values()) / nsteps

    # ---- end to end: host buffers, H2D of the gradients and D2H of the result inside the timing ----
    e2e = None
    if want_e2e and R == M:
        host = torch.empty(R, stride, dtype=w.dtype).pin_memory()
        host.copy_(grads)
        host_out = torch.empty(d, dtype=torch.float32).pin_memory()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(3, min(K, 10))
        copy_stream = torch.cuda.Stream()
        for s in range(reps + 1):
            if s == 1:
                e0.record()
            D.round_trip_from_host(F, host, grads, d, buf, lam, lam_s, 0, 2000 + s, K=w.K, block_log2=b, rank=rank,
                                   world=world, worker_stride=stride, pieces=args.e2e_pieces, copy_stream=copy_stream,
                                   host_out=host_out)
        e1.record()
        barrier()
        t_ms = torch.tensor([e0.elapsed_time(e1) / reps], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(t_ms, op=dist.ReduceOp.MAX)
        e2e = {"value": (M * world) * d / (float(t_ms.item()) * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": R * stride * esize, "d2h_bytes_per_step": d * 4,
               "ms_per_step": float(t_ms.item()), "h2d_pieces": args.e2e_pieces}
        del host, host_out

    # ---- K > 1 on the downlink (server encoder on the finished average + one worker's decoder) ----
    downlink_K = None
    if env["extras"] and world == 1 and want_e2e:
        downlink_K = {}
        for Kd in (1, 3, 7, 15):
            Pd = F.planes(Kd)
            down = torch.zeros(Pd, dp // 32, dtype=torch.int32, device=dev)
            ea, eb, ec = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            reps = 10
            t_enc = t_dec = 0.0
            for r_ in range(reps + 2):
                ea.record()
                F.downlink_encode(buf.acc, d, down, lam_s, 0, 3000 + r_, K=Kd, block_log2=b, ws=ws)
                eb.record()
                F.downlink_decode(down, d, buf.out, lam_s, 0, 3000 + r_, K=Kd, block_log2=b, ws=ws)
                ec.record()
                torch.cuda.synchronize()
                if r_ >= 2:
                    t_enc += ea.elapsed_time(eb)
                    t_dec += eb.elapsed_time(ec)
            downlink_K[str(Kd)] = {"planes": Pd, "server_downlink_encode_ms": t_enc / reps,
                                   "worker_downlink_decode_ms": t_dec / reps,
                                   "encode_algorithmic_GBps": (4 * dp + Pd * dp / 8) / (t_enc / reps) / 1e6,
                                   "decode_algorithmic_GBps": (Pd * dp / 8 + 4 * d) / (t_dec / reps) / 1e6}
            del down

    timeouts = F.async_timeouts()
    rec = {"workload": w, "d": d, "dp": dp, "M": M, "R": R, "P": P, "esize": esize, "n_eff": n_eff,
           "ms_per_step": ms_per_step, "value": value, "steps": K, "repeats": nblocks,
           "block_ms_min_median_max": [min(block_ms), statistics.median(block_ms), max(block_ms)],
           "kernels": kernels, "launches_per_step": launches_per_step, "clocks": clocks, "e2e": e2e,
           "downlink_K": downlink_K, "async_wait_timeouts": timeouts}
    del grads, buf, ws, flush
    torch.cuda.empty_cache()
    return rec


def analyse(rec, peaks, peak_kind, alu_peak, alu_peak_kind, world):
    """Per-call and per-kernel figures of a workload record against the two roofs."""
    w, d, dp, M, R, P, esize = rec["workload"], rec["d"], rec["dp"], rec["M"], rec["R"], rec["P"], rec["esize"]
    kernels, ms_per_step = rec["kernels"], rec["ms_per_step"]
    hbm = peaks["hbm_gbs"]
    chunks = M // R

    def call_ms(pred):
        return sum(v["ms_per_step"] for k, v in kernels.items() if pred(k))

    many = lambda k: not k.endswith("@srv")      # the workers' kernels; "@srv" marks the server's own vector
    up_ms = call_ms(lambda k: is_uplink_kernel(k) and many(k))
    agg_ms = call_ms(lambda k: not is_uplink_kernel(k) and many(k))
    dn_enc_ms = call_ms(lambda k: is_uplink_kernel(k) and "norm" not in k and not many(k))
    dn_dec_ms = call_ms(lambda k: not is_uplink_kernel(k) and not many(k))
    paths = {}

    def path(name, ms, nbytes, extra=None):
        if ms > 0:
            gbs = nbytes / ms / 1e6
            paths[name] = dict({"ms": ms, "algorithmic_bytes": nbytes, "algorithmic_GBps": gbs,
                                "frac_of_hbm_peak": gbs / hbm}, **(extra or {}))

    # the accumulator is read and written once more per extra chunk of streamed workers
    path("uplink_encode", up_ms, M * (d * esize + dp / 8), {"elems_per_s": M * d / up_ms * 1e3 if up_ms else None})
    path("server_decode_average", agg_ms, M * dp / 8 + 4 * dp + 8 * dp * (chunks - 1),
         {"elems_per_s": M * d / agg_ms * 1e3 if agg_ms else None})
    path("server_downlink_encode", dn_enc_ms, 4 * dp + P * dp / 8)
    # every worker computes the same vector: one decode is timed, M of them would run in a deployment
    path("worker_downlink_decode", dn_dec_ms, P * dp / 8 + 4 * d, {"ms_times_workers": dn_dec_ms * M * world})

    per_kernel = {}
    for lab, v in kernels.items():
        if "norm" in lab:
            continue
        t = v["ms_per_launch"] * 1e-3
        alg, impl = algorithmic_bytes(lab, d, dp, P), implementation_bytes(lab, dp, P)
        per_kernel[lab] = {"ms_per_launch": v["ms_per_launch"], "algorithmic_GBps": alg / t / 1e9,
                           "frac": alg / t / 1e9 / hbm, "implementation_GBps": impl / t / 1e9,
                           "implementation_frac": impl / t / 1e9 / hbm}
    dom = max((k for k in kernels if "norm" not in k), key=lambda k: kernels[k]["ms_per_step"])
    _, _, dom_workers = label_parts(dom)
    call_name = ("uplink_encode" if is_uplink_kernel(dom) else "server_decode_average") if many(dom) else \
                ("server_downlink_encode" if is_uplink_kernel(dom) else "worker_downlink_decode")
    call = paths.get(call_name)
    roofline = {"kernel": dom, "bound": "hbm", "unit": "GB/s",
                "achieved": per_kernel[dom]["algorithmic_GBps"], "peak": hbm,
                "frac": per_kernel[dom]["frac"],
                "frac_of_nominal_8TBps": per_kernel[dom]["algorithmic_GBps"] / NOMINAL_HBM_GBS,
                "peak_source": f"{peak_kind} copy bandwidth",
                "traffic": measured_traffic(dom, dom_workers * dp),
                "algorithmic_bytes_per_launch": algorithmic_bytes(dom, d, dp, P),
                "algorithmic_bytes_are": "this launch's share of the method's own traffic (gradients, packed words, "
                                         "accumulator); the fp32/fp16 intermediate between passes is not counted",
                "implementation_bytes_per_launch": implementation_bytes(dom, dp, P),
                "implementation_GBps": per_kernel[dom]["implementation_GBps"],
                "implementation_frac": per_kernel[dom]["implementation_frac"],
                "call": None if call is None else {"name": call_name, "ms": call["ms"],
                                                   "algorithmic_bytes": call["algorithmic_bytes"],
                                                   "achieved": call["algorithmic_GBps"],
                                                   "frac": call["frac_of_hbm_peak"],
                                                   "frac_of_nominal_8TBps": call["algorithmic_GBps"] / NOMINAL_HBM_GBS},
                "per_kernel": per_kernel}
    # the whole step against both roofs, with the algorithmic bytes and operations of the path (per
    # worker-coordinate: the transform's log2 n add/sub plus ~12 for flip, generator, dither and pack
    # on the encode side, ~3 for unpack, flip and accumulate on the decode side; K dithers cost ~9 each)
    Lb = math.log2(rec["n_eff"])
    ops_enc, ops_dec = M * dp * (Lb + 12), M * dp * (Lb + 3)
    ops = ops_enc + ops_dec + dp * (Lb + 3 + 9 * w.K) + dp * (Lb + 3)
    byts = sum(p["algorithmic_bytes"] for p in paths.values())
    t_alu, t_hbm = ops / alu_peak * 1e3, byts / (hbm * 1e9) * 1e3
    path_roofline = {"t_alu_algorithmic_ms": t_alu, "t_hbm_algorithmic_ms": t_hbm,
                     "bound": "alu" if t_alu >= t_hbm else "hbm", "frac": max(t_alu, t_hbm) / ms_per_step,
                     "alu_peak_lane_ops_per_s": alu_peak, "alu_peak_source": alu_peak_kind,
                     "per_call_alu_frac": {
                         "uplink_encode": ops_enc / alu_peak * 1e3 / up_ms if up_ms else None,
                         "server_decode_average": ops_dec / alu_peak * 1e3 / agg_ms if agg_ms else None},
                     "note": "whole step against its algorithmic plain-ALU operation count and byte count"}
    return paths, roofline, path_roofline


def probe_alu(env):
    """Measured issue rates of the plain ALUs (lane operations per second), each kind timed for
    about a third of a second with the SM clock sampled alongside."""
    import torch
    F = env["F"]
    sink = torch.zeros(4, dtype=torch.int32, device=env["dev"])
    kinds = {"fadd": F.PROBE_FADD, "ffma": F.PROBE_FFMA, "lop3": F.PROBE_LOP3, "imad": F.PROBE_IMAD}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(kind, iters):
        e0.record()
        ops = F.probe_issue_rate(kind, iters, sink)
        e1.record()
        torch.cuda.synchronize()
        return ops, e0.elapsed_time(e1) * 1e-3

    out = {}
    sampler = ClockSampler(env["local_rank"])
    seconds = 0.0
    for name, kind in kinds.items():
        timed(kind, 64)
        ops, t = timed(kind, 2048)
        iters = int(max(2048, min(1 << 24, 2048 * 0.35 / t)))
        ops, t = timed(kind, iters)
        seconds += t
        out[name] = ops / t
    clocks = sampler.stop()
    sm_mhz = clocks.get("sm_mhz")
    return {"lane_ops_per_s": out, "seconds_timed": seconds, "clocks": clocks,
            "lanes_per_clock_per_sm": {k: v / (sm_mhz * 1e6 * 148) for k, v in out.items()} if sm_mhz else None,
            "data_sheet_lane_ops_per_s": 148 * 128 * (clocks.get("sm_max_mhz") or 1965.0) * 1e6}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher: start the ranks ourselves (rank 0 prints the line)
        from paper_2405_11095_b200.launch import spawn_ranks
        sys.exit(spawn_ranks([sys.executable, os.path.abspath(__file__), *sys.argv[1:]], args.gpus))
    import torch
    import torch.distributed as dist

    import paper_2405_11095_b200 as F
    from paper_2405_11095_b200 import distributed as D
    from paper_2405_11095_b200 import synthetic

    F.lib()  # fail now if the CUDA library is missing
    if args.fused_encoder:
        F.set_fused_encoder(True)
    if args.tensor_core_pass is not None:
        F.set_tensor_core_pass(args.tensor_core_pass)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    extras = not args.no_legs and world == 1 and args.config == 2 and not args.workers and args.block_log2 == 0
    env = {"F": F, "D": D, "synthetic": synthetic, "dev": dev, "rank": rank, "world": world,
           "local_rank": local_rank, "extras": extras}

    w = synthetic.WORKLOADS[args.config]
    if args.workers:
        w = dataclasses.replace(w, M=args.workers, name=f"{w.name}_workers{args.workers}")
    warmup = max(3, args.warmup)
    rec = run_workload(env, args, w, args.steps, warmup, args.min_seconds, not args.no_e2e)

    # further workloads as sub-records (one GPU, default run only): the ResNet-50-sized and the 1.3B one
    legs = {}
    if extras:
        for cfg, leg_steps, leg_seconds in ((3, 20, 0.5), (4, 3, 0.0)):
            legs[cfg] = run_workload(env, args, synthetic.WORKLOADS[cfg], leg_steps, 3, leg_seconds, False)
    probe = probe_alu(env) if (rank == 0 and not args.no_legs) else None

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = measured_peaks()
    if probe:
        alu_peak, alu_kind = probe["lane_ops_per_s"]["fadd"], "measured fp32-add issue rate (fosgd_probe_issue_rate)"
    else:
        smax = (rec["clocks"] or {}).get("sm_max_mhz") or 1965.0
        alu_peak, alu_kind = 148 * 128 * smax * 1e6, "data sheet: 148 SMs x 128 lanes x max SM clock"
    paths, roofline, path_roofline = analyse(rec, peaks, peak_kind, alu_peak, alu_kind, world)
    dp, P = rec["dp"], rec["P"]
    line = {"metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": rec["ms_per_step"], "repeats": rec["repeats"],
            "block_ms_min_median_max": rec["block_ms_min_median_max"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_config(w, args, world),
            "clocks": rec["clocks"], "e2e": rec["e2e"],
            "gpu_launches": int(round(rec["launches_per_step"] * args.steps)),
            "roofline": roofline, "path_roofline": path_roofline, "paths": paths, "kernels": rec["kernels"],
            "kernel_source_digest": kernel_source_digest(), "async_wait_timeouts": rec["async_wait_timeouts"],
            "path_bytes": {"uplink_bits_per_worker": dp, "downlink_bits": P * dp,
                           "paper_uplink_bits_per_worker": 2 * dp, "paper_downlink_bits": (P + 1) * dp}}
    if rec["downlink_K"]:
        line["downlink_K"] = rec["downlink_K"]
    if probe:
        line["alu_probe"] = probe
    if legs:
        line["legs"] = {}
        for cfg, lr in legs.items():
            lp, lroof, lpr = analyse(lr, peaks, peak_kind, alu_peak, alu_kind, world)
            lw = lr["workload"]
            line["legs"][lw.name] = {"value": lr["value"], "unit": UNIT, "ms_per_step": lr["ms_per_step"],
                                     "steps": lr["steps"], "warmup": 3, "repeats": lr["repeats"],
                                     "config": workload_config(lw, args, world), "clocks": lr["clocks"],
                                     "paths": lp, "kernels": lr["kernels"], "roofline": lroof, "path_roofline": lpr,
                                     "async_wait_timeouts": lr["async_wait_timeouts"]}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = {k: v for k, v in oracle_sample(w, args.block_log2, 2, 0).items()
                                if k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
