#!/usr/bin/env python
"""Benchmark of the implicit-ALS epoch (Gramian -> gather -> normal equations -> solve -> write back, rows then
columns) on synthetic power-law graphs, through the C ABI of libalx_b200.so.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3|cfg2|cfg4|cfg5|medium|small] [--impl ours|reference]

One "step" is one full epoch over the resident graph.  Prints ONE JSON line.  With --impl reference the
fp64 CPU oracle is timed on a bounded sample of the same workload instead (a deliberately slow program:
the ratio to it is context, the roofline fraction is the figure of merit).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from synth import graphs  # noqa: E402

METRIC = "observed entries/sec per ALS epoch"
UNIT = "entries/s"

# the benchmark configurations (synthetic recipe: synth/graphs.py); "cfg3" is the one the headline metric is quoted on
WORKLOADS = {
    "cfg3": dict(n=10_000_000, nnz=1_000_000_000, s=1.1, cap=1_000_000, law="local", delta=100_000, d=128,
                 lam=0.01, alpha=0.001, storage="bf16", seed=0xA1C50003, init_seed=0x1A150003,
                 desc="10M x 10M, 1e9 entries, rank-size Zipf(1.1) degrees (cap 1e6), 80% of a row's entries "
                      "within +-1% of its id, d=128, bf16 tables / fp32 solve"),
    "cfg2": dict(n=1_000_000, nnz=50_000_000, s=1.2, cap=100_000, law="zipf", delta=0, d=64,
                 lam=0.05, alpha=0.001, storage="f32", seed=0xA1C50002, init_seed=0x1A150002,
                 desc="1M x 1M, 5e7 entries, Zipf(1.2) out- and in-degrees (cap 1e5), d=64, fp32 tables"),
    "cfg4": dict(n=50_000_000, nnz=2_000_000_000, s=0.9, cap=2_000_000, law="zipf", delta=0, d=128,
                 lam=0.01, alpha=0.0005, storage="bf16", seed=0xA1C50004, init_seed=0x1A150004,
                 desc="50M x 50M, 2e9 entries, Zipf(0.9) out- and in-degrees (top rows 2e6 entries: split rows), "
                      "d=128, bf16 tables / fp32 solve"),
    "cfg5": dict(n=150_000_000, nnz=5_000_000_000, s=1.1, cap=1_000_000, law="zipf", delta=0, d=128,
                 lam=0.01, alpha=0.0005, storage="bf16", seed=0xA1C50005, init_seed=0x1A150005,
                 desc="150M x 150M, 5e9 entries, Zipf(1.1) degrees (cap 1e6), d=128, bf16 tables (77 GB) plus CSR and "
                      "its transpose (42 GB) resident, 24 GB of chunk sums for the rows longer than 8192 entries"),
    "medium": dict(n=2_000_000, nnz=200_000_000, s=1.1, cap=200_000, law="local", delta=20_000, d=128,
                   lam=0.01, alpha=0.001, storage="bf16", seed=0xA1C500FE, init_seed=0x1A1500FE,
                   desc="2M x 2M, 2e8 entries, scaled-down cfg3 whose tables exceed L2 (profiling case)"),
    "small": dict(n=200_000, nnz=10_000_000, s=1.1, cap=40_000, law="local", delta=2_000, d=128,
                  lam=0.01, alpha=0.001, storage="bf16", seed=0xA1C500FF, init_seed=0x1A1500FF,
                  desc="200k x 200k, 1e7 entries, scaled-down cfg3 (debugging / profiling case)"),
}


def set_initial_table(a, side, w, stream, slice_rows=8_000_000):
    """Initial embeddings of one side, generated on the device in slices (a second full copy of a 38 GB table does
    not fit beside the largest configuration)."""
    from synth import device as sdev
    n = w["n"]
    for r0 in range(0, n, slice_rows):
        cnt = min(slice_rows, n - r0)
        a.set_embedding_rows(side, r0, sdev.device_embeddings(cnt, w["d"], w["init_seed"], stream, w["storage"], row_begin=r0))


def make_spec(w):
    n = w["n"]
    if w["law"] == "local":
        return graphs.GraphSpec(n, n, w["seed"] + 1, law=graphs.LAW_LOCAL, delta=w["delta"])
    if w["law"] == "zipf":
        return graphs.GraphSpec(n, n, w["seed"] + 1, qtable=graphs.zipf_quantile_table(n, w["s"], w["cap"] / w["nnz"]))
    return graphs.GraphSpec(n, n, w["seed"] + 1)


# ----------------------------------------------------------------------------------------------- roofline
def roofline_terms(n, N, nnz, d, e):
    """Algorithmic work of ONE half-epoch: bytes over HBM, tensor flops, FP32-ALU flops."""
    bytes_ = nnz * d * e + nnz * 4 + (n + 1) * 8 + n * 4 + N * d * e + n * d * e
    tensor = 2.0 * nnz * d * d + 2.0 * N * d * d
    alu = n * (d ** 3 / 3.0 + 2.0 * d * d) + 2.0 * nnz * d + n * d * d
    return bytes_, tensor, alu


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi clock / throttle samples during the timed region (read-only queries)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

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
        for r in self.rows:
            try:
                sm.append(float(r[0])); smax.append(float(r[1]))
                for k, nme in enumerate(names):
                    if r[3 + k].lower().startswith("active"):
                        reasons.add(nme)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(w, target_rows, budget_s=None):
    """Time the fp64 oracle on a bounded sample: the first `target_rows` rows of the workload's graph, with the
    fixed table compacted to the columns they touch (Gramian over those rows).  Returns (entries/s, info)."""
    from oracle import ials
    ials.build()
    n, d = w["n"], w["d"]
    spec = make_spec(w)
    deg = graphs.zipf_degrees(n, w["nnz"], w["s"], w["cap"], w["seed"])
    rows = np.arange(min(target_rows, n), dtype=np.int64)
    ptr, cols = graphs.row_columns_flat(spec, rows, deg[rows])
    uniq, inv = np.unique(cols, return_inverse=True)
    from synth import host as synth_host
    X = graphs.storage_to_f64(synth_host.embedding_rows(d, w["init_seed"], 3, w["storage"], rows=uniq), w["storage"])
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    G = ials.gramian(X)
    ials.half_step(ptr, inv.astype(np.int32), None, X, w["alpha"], w["lam"], w["storage"], G=G)
    dt = time.perf_counter() - t0
    nnz_s = int(ptr[-1])
    info = {"kind": "oracle", "cores": cores, "unit": UNIT,
            "sample": f"one half-step over rows 0..{rows.size - 1} of the {w['name']} graph ({nnz_s} entries, "
                      f"{uniq.size} distinct fixed-side rows incl. their Gramian), fp64, OpenMP over rows; "
                      f"{dt:.1f} s; value = sampled entries / seconds (an epoch visits every entry twice, so "
                      f"per-epoch rate is half of this)"}
    # the metric counts entries per EPOCH second; an epoch is two half-steps over the same entries
    return nnz_s / (2.0 * dt), info


# ----------------------------------------------------------------------------------------------- ranks
def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def replica_command(argv, gpus: int, port: int):
    """Command that runs this script as `gpus` replica processes, one per GPU of this node (replicas only: every rank
    runs the whole workload on its own GPU; the ranks meet at the barriers and in the max/sum of the result line)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def aggregate_over_ranks(ms_local: float, units_local: float, world: int, device=None):
    """(max over ranks of the time, sum over ranks of the units) -- replicas only, no data-path collective."""
    if world == 1:
        return ms_local, units_local
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ----------------------------------------------------------------------------------------------- main legs
def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    rows = {"cfg2": 100_000, "small": 30_000, "medium": 30_000}.get(w["name"], 60_000)
    vals = []
    info = None
    for _ in range(args.warmup):
        oracle_sample(w, max(rows // 20, 100))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        v, info = oracle_sample(w, rows)
        vals.append(v)
    ms = (time.perf_counter() - t0) * 1e3 / max(args.steps, 1)
    value = statistics.median(vals)
    info["value"] = value
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": w["name"], "description": w["desc"]},
           "cpu_baseline": info,
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def run_ours(args, w):
    import torch
    from paper_2112_02194_b200 import ALX_COLS, ALX_ROWS, Alx
    from synth import device as sdev
    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    dev = torch.device("cuda", torch.cuda.current_device())
    n, d, storage = w["n"], w["d"], w["storage"]
    e = 2 if storage == "bf16" else 4

    # ---- synthetic inputs, generated on the device (replicas: every rank builds the same graph)
    t_gen = time.perf_counter()
    spec = make_spec(w)
    deg = graphs.zipf_degrees(n, w["nnz"], w["s"], w["cap"], w["seed"])
    rowptr, colidx = sdev.device_csr(spec, deg)
    # the largest configurations leave no room for second copies of the tables and the graph: their tables are
    # generated in slices straight into the context and the end-to-end leg (host copies of everything) is left out
    lean = 2.0 * n * d * e > 32e9
    if lean:
        args.skip_e2e = True
    else:
        W0 = sdev.device_embeddings(n, d, w["init_seed"], 2, storage)
        H0 = sdev.device_embeddings(n, d, w["init_seed"], 3, storage)
    nnz = int(colidx.numel())
    t_gen = time.perf_counter() - t_gen

    a = Alx(n, n, d, w["lam"], w["alpha"], storage=storage, split=w.get("split", 0), solver=args.solver,
            cg_max_iter=args.cg_max_iter, cg_tol=args.cg_tol, cg_start=args.cg_start, dual_cond_limit=args.dual_cond_limit)
    t_set = time.perf_counter()
    a.set_csr(rowptr, colidx)
    torch.cuda.synchronize()
    t_set = time.perf_counter() - t_set
    if lean:
        del colidx
        torch.cuda.empty_cache()
        set_initial_table(a, ALX_ROWS, w, 2)
        set_initial_table(a, ALX_COLS, w, 3)
    else:
        a.set_embeddings(ALX_ROWS, W0)
        a.set_embeddings(ALX_COLS, H0)

    # ---- device-resident timing: K epochs, CUDA events on the context's stream
    for _ in range(args.warmup):
        a.epoch()
    a.synchronize()
    if world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    launches0 = a.get_stats().kernel_launches
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    half_ms = {"rows": [], "cols": [], "gramian": [], "row_kernels": [], "main_kernel": [], "dual_rows": [],
               "cg_rows": [], "cg_products": [], "cg_fallbacks": []}
    ev[0].record()
    trace = []
    for k in range(args.steps):
        for side, key in ((ALX_ROWS, "rows"), (ALX_COLS, "cols")):
            a.half_epoch(side)
            last = k == args.steps - 1
            if args.trace or last:
                # Reading the statistics waits for the stream.  The last timed epoch is read (two waits of a few tens
                # of microseconds between half-epochs of milliseconds): its per-phase CUDA-event times and solver
                # counts are the ones the roofline record uses, taken inside the timed region.  A traced run reads
                # every half-epoch: its epoch times are not bench values.
                s1 = a.get_stats()
                if args.trace:
                    trace.append({"epoch": k, "side": side, "ms": s1.ms_half_epoch, "main_ms": s1.ms_main_kernel,
                                  "cg_rows": s1.cg_rows, "cg_products": s1.cg_products, "cg_fallbacks": s1.cg_fallbacks,
                                  "dual_rows": s1.dual_rows, "cholesky_by_policy": list(s1.cholesky_by_policy)})
                if last:
                    half_ms[key].append(s1.ms_half_epoch)
                    half_ms["gramian"].append(s1.ms_gramian)
                    half_ms["row_kernels"].append(s1.ms_rows)
                    half_ms["main_kernel"].append(s1.ms_main_kernel)
                    half_ms["dual_rows"].append(s1.dual_rows)
                    half_ms["cg_rows"].append(s1.cg_rows)
                    half_ms["cg_products"].append(s1.cg_products)
                    half_ms["cg_fallbacks"].append(s1.cg_fallbacks)
        ev[k + 1].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        torch.distributed.barrier()
    st = a.get_stats()
    launches = st.kernel_launches - launches0
    step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    ms_local = sum(step_ms) / args.steps
    fp32_peak = a.fp32_peak_tflops()
    loss = a.loss()[0]
    evaluation = None
    if args.eval:
        # exact Top-50 of 2048 queries (rows of W) over every row of H, device buffers, outside the timed region
        mq, kq = 2048, 50
        Wq = torch.empty((mq, d), dtype=torch.float32, device=dev)
        a.get_embeddings(ALX_ROWS, row_begin=0, row_count=mq, out=Wq)
        ids_t = torch.empty((mq, kq), dtype=torch.int32, device=dev)
        sc_t = torch.empty((mq, kq), dtype=torch.float32, device=dev)
        t_top = []
        for _ in range(3):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            a.topk_device(ALX_COLS, Wq, kq, ids_t, sc_t)
            torch.cuda.synchronize()
            t_top.append(time.perf_counter() - t0)
        evaluation = {"topk": {"queries": mq, "k": kq, "items": n, "seconds": min(t_top),
                               "scores_per_s": mq * n / min(t_top), "tflops": 2.0 * mq * n * d / min(t_top) / 1e12,
                               "note": "alx_topk on device buffers, best of 3 (includes its scratch allocation and the merge)"}}
    ms, units = aggregate_over_ranks(ms_local, float(nnz), world, dev)
    value = units / (ms * 1e-3)

    # ---- roofline of the dominant phase (the row kernels of one half-epoch)
    peaks = load_peaks()
    b_half, t_half, alu_half = roofline_terms(n, n, nnz, d, e)
    t_bytes = b_half / (peaks["hbm_gbs"] * 1e9)
    t_tensor = t_half / (peaks["bf16_tflops"] * 1e12)
    t_alu = alu_half / (fp32_peak * 1e12)
    t_roof = max(t_bytes, t_tensor + t_alu)
    rows_ms = statistics.mean(half_ms["row_kernels"])
    main_ms = statistics.mean(half_ms["main_kernel"]) or rows_ms
    # dominant kernels: the whole-rows launches (every row of more than 32 and at most 1024 entries, plus the shorter
    # ones when the dual form stepped aside: gather, outer products, solve, store).  Rows and entries per launch are
    # exact: per-class counts from alx_stats minus what the dual-form kernel and the chunks kernel took.
    n_split = [st.rows_in_class[sd][11] for sd in (0, 1)]
    rows_side, ent_side, alu_side = [], [], []
    chol_row = d ** 3 / 3.0 + 3.0 * d * d
    for sd in (0, 1):
        rows_sd = sum(st.rows_in_class[sd][1:11]) - st.long_rows[sd]
        ent_sd = sum(st.entries_in_class[sd][1:11]) - st.long_entries[sd]
        # rows the dual-form kernels took: classes 1 and 2, or class 1 alone where the rows of 17 .. 32 entries went to the
        # whole-rows kernel (alx_stats.dual_rows says which)
        for cl in (1, 2):
            if half_ms["dual_rows"][sd] >= sum(st.rows_in_class[sd][1:cl + 1]) and st.rows_in_class[sd][cl] > 0:
                rows_sd -= st.rows_in_class[sd][cl]
                ent_sd -= st.entries_in_class[sd][cl]
        rows_side.append(rows_sd)
        ent_side.append(ent_sd)
        # solve work of the launch: the cheaper of Cholesky and the products conjugate gradients really spent
        cg_r, cg_p, cg_f = half_ms["cg_rows"][sd], half_ms["cg_products"][sd], half_ms["cg_fallbacks"][sd]
        solve = (rows_sd - cg_r + cg_f) * chol_row + min(cg_r * chol_row, cg_p * (2.0 * d * d + 10.0 * d) + cg_r * d * d)
        alu_side.append(solve + 2.0 * ent_sd * d)
    rows_whole = statistics.mean(rows_side)
    ent_whole = statistics.mean(ent_side)
    alu_main = statistics.mean(alu_side)
    bytes_main = ent_whole * (d * e + 4) + rows_whole * (d * e + 12)
    if t_bytes >= t_tensor + t_alu:
        roof = {"bound": "hbm", "achieved": bytes_main / (main_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "alu", "achieved": alu_main / (main_ms * 1e-3) / 1e12, "peak": fp32_peak, "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    # DRAM traffic of these launches is not measured in this run (it needs a profiler pass); the committed profile
    # summaries hold dram bytes of one capture on the 2M-row `medium` case
    roof["traffic"] = None
    # the half-epoch roofline with the solve counted at what conjugate gradients really spent (never above Cholesky)
    alu_cg_half = statistics.mean([alu_half - rows_side[sd] * chol_row - 2.0 * ent_side[sd] * d + alu_side[sd] for sd in (0, 1)])
    t_alu_cg = alu_cg_half / (fp32_peak * 1e12)
    t_roof_cg = max(t_bytes, t_tensor + t_alu_cg)
    fold = st.kernel_path[0] == 1 and e == 4       # fp32 tables with d = 64 on the tensor cores: split operands
    if st.kernel_path[0] != 1:
        kernel_txt = "k_rows_simple: whole rows on the FP32 ALUs (gather, outer products, Cholesky in shared memory, store)"
    elif fold:
        kernel_txt = ("k_umma<4>: whole rows of 17..512 entries (item gather by TMA from the bfloat16 parts of the fp32 "
                      "table, tcgen05 outer products into tensor memory, fold to the 64 x 64 matrix, conjugate gradients "
                      "on the matrix in registers, Cholesky in shared memory for rows that do not converge, store)")
    else:
        kernel_txt = ("k_umma<3> + k_umma<0>: whole rows (item gather by TMA, tcgen05 outer products into tensor memory, "
                      "conjugate gradients on the matrix in tensor memory, Cholesky in tensor memory for rows that do not "
                      "converge or sides the policy moved, store)")
    short_txt = ("rows with at most 16 entries, solved by k_dual64 outside the dominant kernel" if fold else
                 "rows with at most 32 entries, solved by k_dual outside the dominant kernel")
    long_txt = ("whole rows of more than 512 entries: sums by the chunks kernel, solve by k_solve_sums_fold, outside the "
                "dominant kernel" if fold else
                "whole rows of more than 1024 entries: sums by the chunks kernel, solve by k_solve_sums, outside the "
                "dominant kernel")
    roof.update({"kernel": kernel_txt,
                 "main_kernel_ms": main_ms, "rows_per_launch": rows_whole, "entries_per_launch": ent_whole,
                 "per_side": {"rows": rows_side, "entries": ent_side, "alu_flop": alu_side},
                 "rows_in_dual_form": {"rows": half_ms["dual_rows"][0], "cols": half_ms["dual_rows"][1],
                                       "note": short_txt},
                 "long_rows": {"rows": list(st.long_rows), "entries": list(st.long_entries),
                               "note": long_txt},
                 "peak_source": f"HBM and bf16 {peaks['source']} (sustained bf16); FP32 FMA measured in this run",
                 "half_epoch_ms": {"rows": half_ms["rows"][0], "cols": half_ms["cols"][0],
                                   "gramian": statistics.mean(half_ms["gramian"]), "row_kernels": rows_ms},
                 "roofline_half_epoch_ms": {"bytes": t_bytes * 1e3, "tensor": t_tensor * 1e3, "alu": t_alu * 1e3,
                                            "max(bytes, tensor+alu)": t_roof * 1e3},
                 # mean half-epoch of the timed epochs (the per-phase figures above are the last timed epoch's)
                 "frac_of_roofline_time": t_roof * 1e3 / (0.5 * ms_local),
                 "roofline_half_epoch_ms_solve_as_spent": {"alu": t_alu_cg * 1e3, "max(bytes, tensor+alu)": t_roof_cg * 1e3,
                                                           "frac": t_roof_cg * 1e3 / (0.5 * ms_local),
                                                           "note": "solve counted as min(Cholesky, products x (2d^2 + 10d)) on the rows conjugate gradients took"},
                 "split_rows": n_split})

    # ---- end to end from host buffers: upload S and both tables, one epoch, download both tables
    e2e = None
    cpu_baseline = None
    if args.skip_e2e:
        a.destroy()
    elif rank == 0 or world > 1:
        a.destroy()
        del a
        torch.cuda.empty_cache()
        # a rank that cannot pin its host buffers (8 replicas pin 14 GB each on cfg 3) must not leave the others
        # waiting in the reduction: it reports an infinite time and the line carries no end-to-end figure
        e2e_error = None
        t_e2e = float("inf")
        h2d_bytes = 0
        b = None
        try:
            h_rowptr = torch.empty(rowptr.shape, dtype=rowptr.dtype, pin_memory=True); h_rowptr.copy_(rowptr)
            h_colidx = torch.empty(colidx.shape, dtype=colidx.dtype, pin_memory=True); h_colidx.copy_(colidx)
            np_dt = np.uint16 if storage == "bf16" else np.float32
            view = (lambda t: t.view(torch.int16)) if storage == "bf16" else (lambda t: t)
            h_W = torch.empty(view(W0).shape, dtype=view(W0).dtype, pin_memory=True); h_W.copy_(view(W0))
            h_H = torch.empty(view(H0).shape, dtype=view(H0).dtype, pin_memory=True); h_H.copy_(view(H0))
            del rowptr, colidx, W0, H0
            torch.cuda.empty_cache()
            o_W = torch.empty_like(h_W, pin_memory=True)
            o_H = torch.empty_like(h_H, pin_memory=True)
            b = Alx(n, n, d, w["lam"], w["alpha"], storage=storage, split=w.get("split", 0), solver=args.solver,
                    cg_max_iter=args.cg_max_iter, cg_tol=args.cg_tol, cg_start=args.cg_start, dual_cond_limit=args.dual_cond_limit)
            reps = 2 if w["name"] != "small" else 3
            times = []
            for r in range(reps):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                # upload S and both tables (the tables go over the bus during the set-up kernels), one epoch, both tables
                # back (W during the column pass): the library's two host-buffer calls, both synchronous
                b.load_host(h_rowptr.numpy(), h_colidx.numpy(), None, h_W.numpy().view(np_dt), h_H.numpy().view(np_dt))
                b.epoch_to_host(o_W.numpy().view(np_dt), o_H.numpy().view(np_dt))
                torch.cuda.synchronize()
                times.append(time.perf_counter() - t0)
            t_e2e = min(times[1:]) if len(times) > 1 else times[0]
            h2d_bytes = int(h_rowptr.numel() * 8 + h_colidx.numel() * 4 + 2 * n * d * e)
        except Exception as ex:      # noqa: BLE001 -- reported in the line
            e2e_error = repr(ex)[:300]
            t_e2e = float("inf")
        t_e2e_ms, units_e = aggregate_over_ranks(t_e2e * 1e3, float(nnz), world, dev)
        if not math.isfinite(t_e2e_ms):
            e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                   "error": e2e_error or "the end-to-end leg failed on another rank"}
        else:
            e2e = {"value": units_e / (t_e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d_bytes,
                   "d2h_bytes_per_step": int(2 * n * d * e), "ms_per_step": t_e2e_ms,
                   "covers": "alx_load_host (= alx_set_csr: upload, validate, transpose, degree classes; + both tables, "
                             "uploaded during that work) + alx_epoch_to_host (= alx_epoch + both tables back, W during "
                             "the column pass), pinned host buffers"}
        if b is not None:
            b.destroy()
    if rank == 0 and world == 1 and not args.skip_cpu:
        v, info = oracle_sample(w, {"cfg2": 100_000, "small": 30_000, "medium": 30_000}.get(w["name"], 60_000))
        info["value"] = v
        cpu_baseline = info

    if rank == 0:
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": storage if storage == "bf16" else "f32", "data": "synthetic",
               "config": {"workload": w["name"], "arithmetic": ("bf16 products into f32 sums on the tensor cores, f32 solve"
                                                              if st.kernel_path[0] == 1 else "f32 throughout"), "description": w["desc"], "nnz": nnz, "n_rows": n, "n_cols": n,
                          "d": d, "storage": storage, "lambda": w["lam"], "alpha0": w["alpha"],
                          "step": "one epoch = rows half-epoch + columns half-epoch",
                          "l2": "inputs larger than L2 (tables and index arrays are GBs)",
                          "multi_gpu": "replicas only", "kernel_path": list(st.kernel_path),
                          "paper_context": "about 20 min/epoch for 365M nodes / 29.9B edges on 256 TPU v3 cores"},
               "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roof,
               "cpu_baseline": cpu_baseline,
               "extra": {"evaluation": evaluation, "trace": trace or None, "solver": {"option": args.solver, "cg_rows": half_ms["cg_rows"], "cg_products": half_ms["cg_products"],
                                    "cg_fallbacks": half_ms["cg_fallbacks"],
                                    "note": "[rows half-epoch, columns half-epoch] of the last timed epoch"},
                         "epoch_ms_each": step_ms, "loss_after": loss, "fp32_peak_tflops_measured": fp32_peak,
                         "setup_s": {"generate": t_gen, "alx_set_csr_device": t_set},
                         "rows_in_class": [list(st.rows_in_class[0]), list(st.rows_in_class[1])],
                         "entries_in_class": [list(st.entries_in_class[0]), list(st.entries_in_class[1])],
                         "cholesky_by_policy": list(st.cholesky_by_policy),
                         "n_chunks": list(st.n_chunks), "workspace_gb": st.workspace_bytes / 1e9}}
        print(json.dumps(out))
    if world > 1:
        torch.distributed.destroy_process_group()


def run_cfg1(args):
    """Configuration 1 (2000 x 1500, 40 000 uniform cells, d = 16, fp32 tables): 2.6 MB of data and 2e7 flop per epoch, bound
    by launch latency.  Reported as time per epoch; no roofline is claimed for it."""
    import torch
    from paper_2112_02194_b200 import ALX_COLS, ALX_ROWS, Alx
    torch.cuda.set_device(0)
    rowptr, colidx = graphs.uniform_cells_csr(2000, 1500, 40000, 0xA1C50001)
    W0 = graphs.init_embeddings(2000, 16, 0x1A150001, 2, "f32")
    H0 = graphs.init_embeddings(1500, 16, 0x1A150001, 3, "f32")
    a = Alx(2000, 1500, 16, 0.1, 0.01, storage="f32")
    a.set_csr(rowptr, colidx, None)
    a.set_embeddings(ALX_ROWS, W0)
    a.set_embeddings(ALX_COLS, H0)
    for _ in range(args.warmup):
        a.epoch()
    a.synchronize()
    launches0 = a.get_stats().kernel_launches
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    sampler = ClockSampler(0)
    sampler.start()
    ev[0].record()
    for _ in range(args.steps):
        a.epoch()
    ev[1].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = ev[0].elapsed_time(ev[1]) / args.steps
    launches = a.get_stats().kernel_launches - launches0
    oW, oH = np.empty_like(W0), np.empty_like(H0)
    t0 = time.perf_counter()
    a.load_host(rowptr, colidx, None, W0, H0)
    a.epoch_to_host(oW, oH)
    t_e2e = time.perf_counter() - t0
    a.destroy()
    nnz = int(colidx.size)
    print(json.dumps({"metric": METRIC, "value": nnz / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
                      "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                      "dtype": "f32", "data": "synthetic",
                      "config": {"workload": "cfg1", "description": "2000 x 1500, 40 000 uniform cells, d=16, fp32 tables",
                                 "nnz": nnz, "l2": "fits in L2: latency-bound case, reported as time only"},
                      "clocks": clocks, "gpu_launches": int(launches), "roofline": None, "cpu_baseline": None,
                      "e2e": {"value": nnz / t_e2e, "unit": UNIT, "ms_per_step": t_e2e * 1e3,
                              "h2d_bytes_per_step": int(rowptr.nbytes + colidx.nbytes + W0.nbytes + H0.nbytes),
                              "d2h_bytes_per_step": int(W0.nbytes + H0.nbytes)}}))


def run_cfg1_reference(args):
    """The oracle's whole epoch on configuration 1 (it is small enough to run in full)."""
    if dist_env()[0] != 0:
        return
    from oracle import ials
    ials.build()
    rowptr, colidx = graphs.uniform_cells_csr(2000, 1500, 40000, 0xA1C50001)
    W0 = graphs.init_embeddings(2000, 16, 0x1A150001, 2, "f32").astype(np.float64)
    H0 = graphs.init_embeddings(1500, 16, 0x1A150001, 3, "f32").astype(np.float64)
    for _ in range(args.warmup):
        ials.epoch(rowptr, colidx, None, W0, H0, 0.01, 0.1, "f32")
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ials.epoch(rowptr, colidx, None, W0, H0, 0.01, 0.1, "f32")
    ms = (time.perf_counter() - t0) * 1e3 / max(args.steps, 1)
    value = colidx.size / (ms * 1e-3)
    info = {"kind": "oracle", "cores": os.cpu_count() or 1, "unit": UNIT, "value": value,
            "sample": "the whole epoch of configuration 1 (2000 x 1500, 40 000 entries), fp64, OpenMP over rows"}
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                      "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                      "dtype": "f64", "data": "synthetic", "config": {"workload": "cfg1"}, "cpu_baseline": info,
                      "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=sorted(WORKLOADS) + ["cfg1"])
    ap.add_argument("--solver", type=int, default=0, choices=[0, 1],
                    help="alx_options.solver: 0 = conjugate gradients where available (Cholesky otherwise), 1 = Cholesky")
    ap.add_argument("--cg-max-iter", type=int, default=0, help="alx_options.cg_max_iter (0 = the library's default)")
    ap.add_argument("--cg-start", type=int, default=0, choices=[0, 1],
                    help="alx_options.cg_start: 0 = the stored embedding, 1 = zero")
    ap.add_argument("--cg-tol", type=float, default=0.0, help="alx_options.cg_tol (0 = the library's default)")
    ap.add_argument("--dual-cond-limit", type=float, default=0.0, help="alx_options.dual_cond_limit (0 = the library's default)")
    ap.add_argument("--trace", action="store_true", help="per half-epoch statistics of the timed epochs in extra.trace (perturbs the timing)")
    ap.add_argument("--eval", action="store_true", help="also time the exact Top-K retrieval on the trained tables (extra.evaluation)")
    ap.add_argument("--skip-e2e", action="store_true", help="profiling runs: leave out the host-buffer leg")
    ap.add_argument("--skip-cpu", action="store_true", help="profiling runs: leave out the CPU oracle leg")
    args = ap.parse_args()
    if args.workload == "cfg1":
        return run_cfg1(args) if args.impl == "ours" else run_cfg1_reference(args)
    w = dict(WORKLOADS[args.workload], name=args.workload)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain script: become the launcher of one replica process per GPU
        sys.exit(subprocess.call(replica_command(sys.argv[1:], args.gpus, free_port())))
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
