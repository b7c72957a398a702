#!/usr/bin/env python
"""Throughput of the CHOCO-SGD step (coordinates per second) on synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one call of choco_sgd_step over all n workers: compress x - x^, update the
public copies and neighbour sums, gossip correction and SGD step.  The default workload is
the 8x8-torus, d = 1e6, top-1 % shape.  Prints ONE JSON line.

The path does not shard (one GPU holds all simulated workers), so --gpus N > 1 runs N
independent replicas, one per process, and reports their aggregate.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

L2_BYTES = 126 * 2 ** 20
NOMINAL_HBM_GBS = 8000.0           # the figure the 60 % target is quoted against
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the update kernel, QUOTED from the
# ncu captures summarised under profiles/ (this run does not measure it; None for workloads that
# were not captured, or whose kernel changed since).  The 32-ring QSGD figure is the 8-ring
# capture of the same kernel scaled by the coordinates per launch, as the capture of the
# full-size workload would be too large.
NCU_TRAFFIC = {
    "c4_torus64_topk": (1.3768e9, "profiles/update_and_emit_kernels_c4_torus64_topk.md"),
    "c4_torus64_topk_g004": (1.3768e9, "profiles/update_and_emit_kernels_c4_torus64_topk.md (same kernel and shapes, gamma = 0.2)"),
    "p_ring8_qsgd": (1.9950e9, "profiles/update_dense_bulk_kernel_p_ring8_qsgd.md"),
    "p_ring8_sign": (1.8544e9, "profiles/update_dense_bulk_kernel_p_ring8_sign.md"),
    "c5_ring32_qsgd": (29.73 * 32 * 25_557_032,
                       "profiles/update_dense_bulk_kernel_p_ring8_qsgd.md (the 8-ring capture of the same kernel, "
                       "29.73 B per coordinate, scaled by the coordinates per launch)"),
}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------
# byte model: what one step must move (each dense array once, messages once per reader)
# ------------------------------------------------------------------------------------------


def message_bytes_of(q: str, d: int, k: int, s: int, bucket: int) -> int:
    if q == "topk":
        return 8 * k
    if q == "randk":
        return 4 * k
    if q == "sign":
        return 4 * ((d + 31) // 32) + 4
    if q == "qsgd":
        blen = bucket or d
        wbits = 1
        while (1 << wbits) < s:
            wbits *= 2
        return 4 * ((d + blen - 1) // blen) + 4 * ((d + 31) // 32) + (d * wbits + 7) // 8
    return 4 * d


def layer_k(wl, length: int) -> int:
    return max(1, (length * wl.a_num) // wl.a_den)


def entries_per_row(wl) -> int:
    """Entries a sparse Q keeps per worker (summed over the layers, if any)."""
    if wl.layers:
        return sum(layer_k(wl, dl) for dl in wl.layer_sizes())
    return wl.k


def message_bytes(wl) -> int:
    """Per worker and step, by the paper's accounting."""
    if wl.layers:
        return sum(message_bytes_of(wl.q, dl, layer_k(wl, dl), wl.s, wl.bucket) for dl in wl.layer_sizes())
    return message_bytes_of(wl.q, wl.d, wl.k, wl.s, wl.bucket)


def step_min_bytes(wl, w, sgd=True) -> int:
    """Whole step: X, Xhat, S (and G) read once, every densely changing array written once,
    messages written once and read once per off-diagonal neighbour, sparse updates at 4 B;
    Algorithm 2 reads and writes the momentum memory as well (8 B per coordinate)."""
    if wl.momentum > 0:
        return step_min_bytes(dataclasses.replace(wl, momentum=0.0), w, sgd) + 8 * wl.n * wl.d
    N = wl.n * wl.d
    nnz = int(w.row_ptr[-1])
    deg_off = nnz - wl.n
    msg = message_bytes(wl)
    if wl.q in ("topk", "randk"):
        dense = (20 if sgd else 16) * N
        k = entries_per_row(wl)
        return dense + msg * wl.n + msg * deg_off + 4 * (wl.n * k + nnz * k)
    dense = (28 if sgd else 24) * N
    return dense + msg * wl.n + msg * deg_off


def update_kernel_bytes(wl, w, sgd=True) -> int:
    """The update kernel alone: reads X, Xhat, S, G and every neighbour's message (self
    included), writes X densely and Xhat, S where touched (all of them for dense Q); with
    momentum (Algorithm 2) M is read and written too."""
    if wl.momentum > 0:
        return update_kernel_bytes(dataclasses.replace(wl, momentum=0.0), w, sgd) + 8 * wl.n * wl.d
    N = wl.n * wl.d
    nnz = int(w.row_ptr[-1])
    msg = message_bytes(wl)
    if wl.q in ("topk", "randk"):
        per_entry = 8                                   # index + value as read by the kernel
        k = entries_per_row(wl)
        return (20 if sgd else 16) * N + per_entry * k * nnz + 4 * (wl.n * k + nnz * k)
    return (28 if sgd else 24) * N + msg * nnz


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15 and len(r) >= 6] or \
               [r for _, r in self.rows if len(r) >= 6]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        mhz = sorted(float(r[0]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[2 + i].lower().startswith("active") for r in rows)]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": float(rows[0][1]), "reasons": reasons,
                "samples": len(rows)}


# ------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands (baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------


def oracle_sample(wl, w, budget_rows=None):
    """Time the oracle, as it stands and on one thread, on a row sample of the workload, and
    build the time of a WHOLE step from it: a step forms n messages and updates n rows, so
    step seconds = n * (seconds per message + seconds per row update), both measured here
    (the sample updates `rows` rows and has to form the messages of all their neighbours, which
    are more; each cost is divided by its own count).  Returns (seconds per whole step, seconds
    spent, text)."""
    import oracle
    rows = list(range(wl.n)) if budget_rows is None else list(range(min(budget_rows, wl.n)))
    need = sorted({int(c) for i in rows for c in w.col[w.row_ptr[i]:w.row_ptr[i + 1]]})
    remap = {j: a for a, j in enumerate(need)}
    X = workloads.normal_rows(len(need), wl.d, wl.x_var or 1.0, 11)
    Xh, S = np.zeros_like(X), np.zeros_like(X)
    G = workloads.normal_rows(len(need), wl.d, wl.g_var or 1e-2, 12)
    M = np.zeros_like(X) if wl.momentum > 0 else None
    # a sub-problem holding only the needed rows, W's rows restricted accordingly
    rp, col, val = [0], [], []
    for j in need:
        if j in rows:
            for e in range(w.row_ptr[j], w.row_ptr[j + 1]):
                col.append(remap[int(w.col[e])]); val.append(float(w.val[e]))
        else:
            col.append(remap[j]); val.append(1.0)
        rp.append(len(col))
    sub = workloads.MixingCSR(len(need), np.asarray(rp, np.int32), np.asarray(col, np.int32),
                              np.asarray(val, np.float32))
    p = oracle.Params(wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=1)
    # a stop-watch around the oracle's compression call: everything else a step does is the row update
    spent = {"compress": 0.0}
    plain_compress = oracle.compress

    def timed_compress(*a, **kw):
        t = time.perf_counter()
        out = plain_compress(*a, **kw)
        spent["compress"] += time.perf_counter() - t
        return out

    oracle.compress = timed_compress
    try:
        t0 = time.perf_counter()
        if wl.layers:
            oracle.step_layers(sub, p, workloads.layer_offsets(wl.layer_sizes()), wl.a_num, wl.a_den, X, Xh, S, G,
                               wl.eta, wl.gamma, 0, rows=[remap[i] for i in rows], M=M, lam=wl.weight_decay,
                               beta=wl.momentum)
        else:
            oracle.step(sub, p, X, Xh, S, G, wl.eta, wl.gamma, 0, rows=[remap[i] for i in rows], M=M,
                        lam=wl.weight_decay, beta=wl.momentum)
        dt = time.perf_counter() - t0
    finally:
        oracle.compress = plain_compress
    per_msg = spent["compress"] / len(need)
    per_row = (dt - spent["compress"]) / len(rows)
    text = (f"whole step of {wl.name} built from measured costs: n * (per message + per row update), "
            f"{per_msg:.4f} s per message over {len(need)} messages and {per_row:.4f} s per row update over "
            f"{len(rows)} of {wl.n} rows, oracle as it stands, single thread")
    return wl.n * (per_msg + per_row), dt, text


def rows_for_budget(wl, seconds=20.0) -> int:
    # ~0.15 s per million coordinates compressed + applied; a sparse Q sorts the row (3x)
    per_row = 0.25 * wl.d / 1e6 * (3 if wl.q in ("topk", "randk") else 1)
    return max(1, min(wl.n, int(seconds / max(per_row, 1e-3))))


# ------------------------------------------------------------------------------------------


def max_over_ranks(values, device):
    """The slowest rank's figure for each entry: every replica must have finished."""
    import torch
    import torch.distributed as dist
    tt = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return [float(v) for v in tt]


def whole_job_rate(world: int, coords_per_replica_step: int, steps: int, seconds: float) -> float:
    """Coordinates per second over all replicas: each of `world` ranks ran `steps` steps."""
    return world * coords_per_replica_step * steps / seconds


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="c4_torus64_topk", choices=sorted(workloads.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--repeats", type=int, default=5, help="timed regions of --steps steps each; the median is reported")
    ap.add_argument("--kernel-launches", type=int, default=32,
                    help="launches of the update kernel timed one by one after the timed regions")
    ap.add_argument("--pool", type=int, default=8, help="gradient tensors cycled through (>= 2)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.repeats = max(args.repeats, 1)
    args.kernel_launches = max(args.kernel_launches, 16)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = workloads.WORKLOADS[args.workload]
    w = wl.mixing()
    N = wl.n * wl.d
    config = {"workload": wl.name, "n": wl.n, "d": wl.d, "graph": wl.graph, "Q": wl.q,
              "k": entries_per_row(wl) if wl.q in ("topk", "randk") else 0, "s": wl.s, "bucket": wl.bucket,
              "layers": (f"{wl.layers}: Q per layer, {len(wl.layer_sizes())} layers" if wl.layers else "none: Q on the whole row"),
              "eta": wl.eta, "gamma": wl.gamma,
              "parallelism": "replicas only" if args.gpus > 1 else "single GPU",
              "l2": "inputs per step exceed L2" if 20 * N > 2 * L2_BYTES else "state fits L2 (no flush)"}

    host_cores = os.cpu_count()
    if args.impl == "reference":
        if rank != 0:
            return
        # every timed step is a whole step of the stated workload, its time built from a bounded
        # sample (see oracle_sample); the whole run is sized to about two minutes
        rows = rows_for_budget(wl, 120.0 / (args.steps + args.warmup))
        step_s, text = [], ""
        for i in range(args.warmup + args.steps):
            sec, _, text = oracle_sample(wl, w, rows)
            if i >= args.warmup:
                step_s.append(sec)
        mean_s = sum(step_s) / len(step_s)
        val = N / mean_s
        print(json.dumps({
            "impl": "reference", "metric": "coords_per_sec", "value": val, "unit": "coords/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * mean_s, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": val, "unit": "coords/s", "cores": 1, "host_cores": host_cores,
                             "kind": "oracle", "sample": text},
            "e2e": {"value": val, "unit": "coords/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return

    import torch
    import torch.distributed as dist
    import paper_1907_09356_b200 as choco

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    small = N <= (1 << 22)      # the library replays such problems' steps from CUDA graphs
    if wl.layers or small:
        # a stream that can be captured: steady-state steps are replayed from CUDA graphs,
        # which the legacy default stream does not allow
        torch.cuda.set_stream(torch.cuda.Stream(device=dev))

    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)
    X = torch.randn(wl.n, wl.d, device=dev, generator=gen) * float(np.sqrt(wl.x_var or 1.0))
    Xh = torch.zeros_like(X)
    S = torch.zeros_like(X)
    free_b = torch.cuda.mem_get_info(dev)[0]
    pool_n = int(max(2, min(args.pool, (free_b * 0.5) // (4 * N))))
    if small:
        pool_n = 2                  # the state fits L2 anyway; fewer argument sets to capture
    if wl.layers or small:
        # graph replay: an argument set (gradient tensor x message-buffer parity) runs kernel by
        # kernel when first seen and is captured when seen again; the warm-up covers both
        args.warmup = max(args.warmup, 4 * pool_n + 2)
    pool = [torch.randn(wl.n, wl.d, device=dev, generator=gen) * float(np.sqrt(wl.g_var or 1e-2))
            for _ in range(pool_n)]
    mom = wl.momentum > 0
    M = torch.zeros_like(X) if mom else None
    if wl.layers:
        off = workloads.layer_offsets(wl.layer_sizes())
        lay = choco.choco_layers_init(wl.n, off, wl.d, w.row_ptr, w.col, w.val, wl.q, wl.a_num, wl.a_den,
                                      s=wl.s or 16, bucket=wl.bucket, seed=7)
        ctxs = [choco.choco_layers_get_layer(lay, l)[0] for l in range(len(off) - 1)]

        def do_step(G):
            if mom:
                choco.choco_layers_sgd_momentum_step(lay, X, Xh, S, G, M, wl.eta, wl.gamma, wl.weight_decay,
                                                     wl.momentum)
            else:
                choco.choco_layers_sgd_step(lay, X, Xh, S, G, wl.eta, wl.gamma)
    else:
        ch = choco.Choco(w, wl.d, wl.q, k=wl.k, s=wl.s or 16, bucket=wl.bucket, seed=7)
        ctxs = [ch.ctx]

        def do_step(G):
            if mom:
                ch.sgd_momentum_step(X, Xh, S, G, M, wl.eta, wl.gamma, wl.weight_decay, wl.momentum)
            else:
                ch.sgd_step(X, Xh, S, G, wl.eta, wl.gamma)

    def stats_sum():
        tot = {}
        for c in ctxs:
            for key, v in choco.choco_get_stats(c).items():
                tot[key] = tot.get(key, 0) + int(v)
        return tot

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(args.warmup):
        do_step(pool[t % pool_n])
    barrier()
    st0 = stats_sum()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    # the timed region, EXACTLY --steps steps between a barrier + synchronize on both sides, taken
    # --repeats times back to back; the line reports the median repeat (and the fastest beside it)
    t_wall0 = time.time()
    step_no = args.warmup
    rep_ms = []
    for _ in range(args.repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for t in range(args.steps):
            do_step(pool[step_no % pool_n])
            step_no += 1
        e1.record()
        barrier()
        rep_ms.append(e0.elapsed_time(e1))
    st1 = stats_sum()
    # the dominant kernel by itself: CUDA events around the update kernel on the step's stream, on
    # every one of a few further steps (outside the timed region: events between a step's kernels
    # keep them from overlapping and would slow the steps down)
    nrec, upd_ms = 0, 0.0
    if not wl.layers and not small:
        choco.choco_profile_enable(ch.ctx, args.kernel_launches)
        for t in range(args.kernel_launches):
            do_step(pool[step_no % pool_n])
            step_no += 1
        nrec, upd_ms = choco.choco_profile_read(ch.ctx)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    finite = bool(torch.isfinite(X).all())

    # end to end: host buffers in, host buffers out, through choco_sgd_step_host
    e2e = None
    if args.e2e_steps > 0:
        hX, hXh, hS = (t.cpu().pin_memory() for t in (X, Xh, S))
        hG = pool[0].cpu().pin_memory()
        hM = M.cpu().pin_memory() if mom else None
        if wl.layers or mom:
            # these calls take device arrays: copy in from pinned memory, step, copy out
            def host_step():
                for dst, src in ((X, hX), (Xh, hXh), (S, hS), (pool[0], hG)) + (((M, hM),) if mom else ()):
                    dst.copy_(src, non_blocking=True)
                for c in ctxs:
                    choco.choco_invalidate(c)      # the arrays were overwritten behind the library's back
                do_step(pool[0])
                for dst, src in ((hX, X), (hXh, Xh), (hS, S)) + (((hM, M),) if mom else ()):
                    dst.copy_(src, non_blocking=True)
                torch.cuda.synchronize()
        else:
            def host_step():
                choco.choco_sgd_step_host(ch.ctx, hX, hXh, hS, hG, wl.eta, wl.gamma)
        host_step()                                                # warm-up, allocates staging
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            host_step()
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        e2e = {"seconds": e2e_s, "steps": args.e2e_steps}

    if world > 1:
        got = max_over_ranks(rep_ms + [e2e["seconds"] if e2e else 0.0], dev)
        rep_ms = got[:-1]
        if e2e:
            e2e["seconds"] = got[-1]

    if rank == 0:
        peak, peak_src = measured_peak()
        ms = sorted(rep_ms)[len(rep_ms) // 2]           # the median repeat
        ms_step = ms / args.steps
        value = whole_job_rate(world, N, args.steps, ms * 1e-3)
        upd_bytes = update_kernel_bytes(wl, w)
        upd_avg_s = (upd_ms / max(nrec, 1)) * 1e-3
        achieved = upd_bytes / upd_avg_s / 1e9 if nrec else None
        step_bytes = step_min_bytes(wl, w)
        step_gbs = step_bytes / (ms_step * 1e-3) / 1e9
        roof_kernel = "update (apply) kernel"
        if wl.layers or small:
            # a few short kernels replayed from a graph (events between them would prevent that):
            # no single dominant launch to time, so the roofline entry is the whole step against
            # its minimum bytes
            roof_kernel = ("whole step: the kernels of all layers" if wl.layers
                           else "whole step (state fits L2; replayed from a CUDA graph)")
            achieved, upd_bytes, upd_avg_s, nrec = step_gbs, step_bytes, ms_step * 1e-3, args.steps
        traffic, traffic_src = NCU_TRAFFIC.get(wl.name, (None, None))
        out = {
            "metric": "coords_per_sec", "value": value, "unit": "coords/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config,
            "repeats": {"count": len(rep_ms), "ms_per_step": [m / args.steps for m in rep_ms],
                        "median_ms_per_step": ms_step, "min_ms_per_step": min(rep_ms) / args.steps,
                        "reported": "median"},
            "steps_per_sec": 1e3 / ms_step,
            "compressed_bytes_per_step": message_bytes(wl) * wl.n,
            "step_min_bytes": step_bytes, "step_hbm_gbs": step_gbs,
            "step_frac_of_measured_peak": step_gbs / peak,
            "step_frac_of_nominal_8tbs": step_gbs / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "kernel": roof_kernel, "achieved": achieved,
                         "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                         "frac": (achieved / peak) if achieved else None,
                         "traffic": traffic,
                         "traffic_source": (f"quoted from the ncu capture in {traffic_src}, not measured by this run"
                                            if traffic_src else None),
                         "algorithmic_bytes_per_launch": upd_bytes,
                         "avg_launch_ms": upd_avg_s * 1e3, "launches_timed": nrec},
            "gpu_launches": int(st1["kernel_launches"] - st0["kernel_launches"]),
            "selection": {k: int(st1[k] - st0[k]) for k in ("prepared_rows", "recompressed_rows", "exact_rows",
                                                          "rescued_rows")},
            "finite": finite,
            "clocks": clocks,
        }
        if wl.layers:
            out["graph_replays"] = int(choco.choco_layers_set_graphs(lay))
        else:
            out["graph_replays"] = int(st1["graph_replays"] - st0["graph_replays"])
        if e2e:
            arrays_in, arrays_out = (5, 4) if mom else (4, 3)
            out["e2e"] = {"value": whole_job_rate(world, N, e2e["steps"], e2e["seconds"]), "unit": "coords/s",
                          "h2d_bytes_per_step": 4 * arrays_in * N, "d2h_bytes_per_step": 4 * arrays_out * N,
                          "steps": e2e["steps"],
                          "api": ("pinned host buffers copied in and out around the device-pointer step call"
                                  if (wl.layers or mom) else "choco_sgd_step_host, pinned host buffers")}
        if not args.no_cpu_baseline and world == 1:
            step_s, dt, text = oracle_sample(wl, w, rows_for_budget(wl))
            out["cpu_baseline"] = {"value": N / step_s, "unit": "coords/s", "cores": 1, "host_cores": host_cores,
                                   "kind": "oracle", "sample": text, "seconds": dt}
        print(json.dumps(out))
    if wl.layers:
        choco.choco_layers_destroy(lay)
    else:
        ch.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
