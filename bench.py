#!/usr/bin/env python
"""Benchmark of the sampled-GNN training pass (sample -> forward -> backward) on B200.

One step = k-hop sampling of one seed batch, the GraphSAGE forward over the sampled blocks and the
full backward (weight gradients and feature-row gradients), through the library's C ABI.  Prints one
JSON line (rank 0).

Without --workload the line is the `large` workload (the largest configuration that fits one GPU) and
carries, as sub-records, the `medium` workload, the joint step (encoder + ranking tower) on the medium
graph and the whole-graph aggregation, each with its own roofline block.  With --workload only that
workload runs.  `--impl reference` times the CPU oracle instead (a deliberately plain program).
"""
from __future__ import annotations

import argparse
import gc
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as S  # noqa: E402

METRIC = "sampled_gnn_sample_fwd_bwd_edges_per_sec"
UNIT = "edges/s"
NOMINAL_HBM_GBS = 8000.0            # the ~8 TB/s figure of the hardware's data sheet; fractions are given against it and the measured copy peak
MIN_TIMED_S = 0.5                   # the K-step loop is repeated until the timed region is at least this long
CLOCK_QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
TAP_NAMES = {1: "layer-0 mean aggregation (sage_aggregate_kernel; sage_aggregate_stream_kernel where the block can hold 2^20 entries or more)",
             2: "seg_run_block_kernel (layer-0 transposed aggregation -> dX rows)",
             3: "layer-0 dense transform W[h|agg]",
             4: "layer-0 weight gradient dZ^T[h|agg]",
             5: "layer-0 input gradient dZ W",
             6: "e2egrec_sample_khop (all sampling kernels)",
             7: "seg_run_block_kernel, top layer (first transposed aggregation of the backward pass)",
             9: "seg_final_kernel (same; empty interval where the one-launch form runs)"}
# source files whose kernels a recorded DRAM-traffic figure belongs to (the figure is dropped when they change)
TRAFFIC_SOURCES = ("aggregate.cuh", "segreduce.cuh", "common.cuh", "gather_stream.cu")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    sm_max_mhz=float(d.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


def fp32_alu_peak_tflops(peaks):
    """Plain fp32 FMA peak: 148 SMs x 128 fp32 lanes x 2 flop per FMA x the maximum SM clock (74.4 TFLOP/s at 1965 MHz)."""
    return 148 * 128 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12


def source_digest():
    h = hashlib.sha256()
    for name in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, "paper_2511_20564_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(key):
    """DRAM bytes (read + write) per unit of work of one ncu capture, recorded in profiles/traffic.json beside the
    summary it came from; None when there is no record or the kernel sources have changed since the capture."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(p):
        return None
    rec = json.load(open(p)).get(key)
    if not rec or rec.get("source_sha") != source_digest():
        return None
    return rec


class ClockSampler:
    """SM clock and clock-event reasons read DURING the timed region.  NVML is polled from a thread every few
    milliseconds (read-only queries), so even a region of tens of milliseconds holds several samples; without
    the NVML module the same fields come from an `nvidia-smi -lms` child process."""
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index, period_s=0.004):
        self.gpu = gpu_index
        self.period = period_s
        self.rows = []                  # (time.time(), sm MHz, max sm MHz, [reason names])
        self.thread = self.p = self.nv = None
        self.stop_flag = False
        self.path = f"/tmp/e2egrec_clocks_{os.getpid()}.csv"

    def _nvml_handle(self):
        import pynvml
        import torch
        pynvml.nvmlInit()
        try:
            uuid = str(torch.cuda.get_device_properties(self.gpu).uuid)
            return pynvml, pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            ids = [v for v in vis.split(",") if v.strip().isdigit()]
            return pynvml, pynvml.nvmlDeviceGetHandleByIndex(int(ids[self.gpu]) if self.gpu < len(ids) else self.gpu)

    def _poll(self):
        nv, h = self.nv
        bits = [nv.nvmlClocksEventReasonHwSlowdown, nv.nvmlClocksEventReasonHwThermalSlowdown,
                nv.nvmlClocksEventReasonSwThermalSlowdown, nv.nvmlClocksEventReasonSwPowerCap]
        smax = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
        while not self.stop_flag:
            try:
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                sm = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                self.rows.append((time.time(), sm, smax, [n for n, b in zip(self.NAMES, bits) if mask & b]))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        try:
            self.nv = self._nvml_handle()
            import threading
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nv = self.thread = None
        try:
            self.f = open(self.path, "w")
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={CLOCK_QUERY}",
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def mark(self):
        return time.time()

    def _smi_rows(self):
        import datetime
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.close()
        for line in open(self.path):
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.rows.append((ts, float(c[1]), float(c[2]),
                                  [n for n, v in zip(self.NAMES, c[5:9]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        try:
            os.remove(self.path)
        except OSError:
            pass

    def stop(self, t_begin=None, t_end=None):
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            source, slack = "nvml", 0.0
        elif self.p is not None:
            self._smi_rows()
            source, slack = "nvidia-smi", 0.05
        else:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no clock source"], samples=0)
        rows = [r for r in self.rows if t_begin is None or t_begin - slack <= r[0] <= t_end + slack]
        sm, smax = [r[1] for r in rows], [r[2] for r in rows]
        reasons = sorted({n for r in rows for n in r[3]})
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=reasons, samples=len(sm), source=source)


def hbm_fractions(gbs, peaks):
    return dict(gbs=gbs, frac_of_measured_copy=gbs / peaks["hbm_gbs"], frac_of_nominal_8tbs=gbs / NOMINAL_HBM_GBS)


def build_inputs(w: S.Workload, host_csr=True):
    """Interactions, features and weights; the host CSR (numpy) is only built for the CPU oracle."""
    users, items = S.bipartite_interactions(w.n_users, w.n_items, w.n_interactions, w.alpha_user, w.alpha_item,
                                            w.seed, w.q)
    indptr = indices = None
    if host_csr:
        row, col = S.undirected_coo(users, items)
        indptr, indices = S.coo_to_csr(w.n_nodes, row, col)
    X, Ws = S.build_model(w)
    return indptr, indices, X, Ws, (users, items)


def make_batches(w, inter, recipe, first, count):
    """Seed batches for steps first .. first+count-1: `activity` draws nodes as endpoints of random
    interactions (the source nodes of a training stream), `uniform` draws them uniformly over all ids."""
    if recipe == "uniform":
        return np.stack([S.seed_batch(w.n_nodes, w.batch, w.seed, first + i) for i in range(count)])
    return np.stack([S.seed_batch_from_interactions(inter[0], inter[1], w.batch, w.seed, first + i)
                     for i in range(count)])


def upstream_grad(w, rows):
    g = np.random.default_rng(4321).standard_normal((rows, w.hidden)).astype(np.float32)
    return S.to_bf16_values(g) if w.dtype == "bf16" else g


def on_device_workload(w):
    """Graphs of 10^8 interactions and more are drawn with torch on the GPU that will hold them (the host arrays
    alone would take minutes and tens of GB)."""
    return w.n_interactions >= 100_000_000


# ------------------------------------------------------------------------------------------ the CPU oracle, timed
def oracle_step(w, indptr, indices, X, Ws, seeds, step, dH, edge_cum=None):
    """One oracle step.  X is the host feature table, or a callable ids -> rows (table kept elsewhere)."""
    import oracle
    bf16 = w.dtype == "bf16"
    blocks = oracle.sample_khop(indptr, indices, seeds, w.fanouts, w.seed, step, edge_cum=edge_cum)
    if callable(X):
        out, ctx = oracle.sage_forward(blocks, X(blocks[-1]["src_nodes"]), Ws, bf16=bf16, gathered=True)
    else:
        out, ctx = oracle.sage_forward(blocks, X, Ws, bf16=bf16)
    oracle.sage_backward(blocks, ctx, Ws, dH[: seeds.size], bf16=bf16)
    return sum(b["n_edges"] for b in blocks)


def time_oracle(step_fn, budget_s, max_steps, unit, describe):
    """The oracle as it stands on all host cores (its row loops carry OpenMP pragmas) and on one: `step_fn(i)` runs
    step i and returns the units of work it did.  Returns the cpu_baseline record (value = the all-core figure)."""
    import oracle
    out = {}
    all_cores = oracle.max_threads()
    for label, threads in (("all", all_cores), ("one", 1)):
        oracle.set_threads(threads)
        t0 = time.perf_counter()
        work, n = 0, 0
        while n < max_steps and (n == 0 or time.perf_counter() - t0 < budget_s):
            work += step_fn(n)
            n += 1
        dt = time.perf_counter() - t0
        out[label] = dict(value=work / dt, steps=n, seconds=dt)
    oracle.set_threads(all_cores)
    return dict(value=out["all"]["value"], unit=unit, cores=all_cores, kind="oracle",
                sample=describe(out["all"]["steps"], out["all"]["seconds"]),
                single_core=dict(value=out["one"]["value"], unit=unit, cores=1,
                                 sample=describe(out["one"]["steps"], out["one"]["seconds"])),
                host_cores=os.cpu_count())


def reference_workload(w):
    """The CPU arm runs the device-drawn workloads on a 1/100-scale graph of the same recipe."""
    if not on_device_workload(w):
        return w, ""
    import dataclasses
    small = dataclasses.replace(w, n_users=w.n_users // 100, n_items=w.n_items // 100,
                                n_interactions=w.n_interactions // 100, q=w.q / 100)
    return small, " on a 1/100-scale graph of the same recipe"


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    import oracle
    oracle.build()
    w, scale_note = reference_workload(w)
    indptr, indices, X, Ws, inter = build_inputs(w)
    cum = None
    if args.beta is not None:
        cum = oracle.edge_cumulate(indptr, S.edge_weight_units(indptr, w.seed, args.beta))
    sample = args.ref_seeds
    dH = upstream_grad(w, sample).astype(np.float64)
    batches = make_batches(w, inter, args.seeds, 0, args.warmup + args.steps)[:, :sample]
    cores = oracle.max_threads()
    for i in range(args.warmup):
        oracle_step(w, indptr, indices, X, Ws, batches[i], i, dH, cum)
    t0 = time.perf_counter()
    edges = 0
    for i in range(args.warmup, args.warmup + args.steps):
        edges += oracle_step(w, indptr, indices, X, Ws, batches[i], i, dH, cum)
    dt = time.perf_counter() - t0
    val = edges / dt
    desc = f"first {sample} of the {w.batch} seeds of each step's batch, full sample+forward+backward{scale_note}"
    return dict(impl="reference", metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=dt / args.steps * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=w.name, nodes=w.n_nodes, csr_entries=int(indptr[-1]), dim=w.dim, hidden=w.hidden,
                            layers=len(w.fanouts), fanouts=list(w.fanouts), batch=w.batch, seeds=args.seeds,
                            sample=desc),
                cpu_baseline=dict(value=val, unit=UNIT, cores=cores, kind="oracle", sample=desc),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)


# ------------------------------------------------------------------------------------------ our arm
def run_ours(args, w, with_joint):
    import torch
    import torch.distributed as dist
    import paper_2511_20564_b200 as E

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    E.lib()                                            # fails loudly if the CUDA library is missing

    want_cpu = world == 1 and not args.no_cpu_baseline
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    K, Wm = args.steps, args.warmup
    total = K + Wm + 4                                 # + the batches whose sampling / upload is prefetched during the last steps
    first_step = rank * 1_000_000                      # = replicas.first_step_of(rank)
    on_device = on_device_workload(w)
    t_setup = time.perf_counter()
    if on_device:
        users_d, items_d = S.bipartite_interactions_device(w.n_users, w.n_items, w.n_interactions, w.alpha_user,
                                                           w.alpha_item, w.seed, w.q, dev)
        row_d, col_d = torch.cat([users_d, items_d]), torch.cat([items_d, users_d])
        indptr_h = indices_h = X_h = None
        Ws_h = S.build_weights(w)
        inter = None
    else:
        indptr_h, indices_h, X_h, Ws_h, inter = build_inputs(w, host_csr=want_cpu)
        row_d = torch.cat([torch.from_numpy(inter[0]), torch.from_numpy(inter[1])]).to(dev)
        col_d = torch.cat([torch.from_numpy(inter[1]), torch.from_numpy(inter[0])]).to(dev)
    # graph ingest on the device: both directions of every interaction -> canonical CSR
    indptr, indices, ingest_status = E.graph_from_coo(w.n_nodes, row_d, col_d)
    indices = indices.contiguous()
    if int(ingest_status):
        raise RuntimeError("graph ingest: node id out of range")
    del row_d, col_d
    torch.cuda.empty_cache()
    edge_cum = q_h = None
    if args.beta is not None:
        if on_device:
            raise SystemExit("--beta is not wired for workloads drawn on the device")
        # importance sampling p ~ omega^beta (Sec. 4.1): integer weights drawn from the row lengths alone, running sums on the device
        deg_h = np.bincount(np.concatenate([inter[0], inter[1]]), minlength=w.n_nodes)
        ip_h = np.zeros(w.n_nodes + 1, np.int64)
        np.cumsum(deg_h, out=ip_h[1:])
        q_h = S.edge_weight_units(ip_h, w.seed, args.beta)
        edge_cum = E.edge_cumulate(indptr, torch.from_numpy(q_h.view(np.int32)).to(dev))
    # every rank trains on its own batches (data parallel replicas; no exchange on the measured path)
    if on_device:
        if args.seeds == "uniform":
            seeds_h = np.stack([S.seed_batch(w.n_nodes, w.batch, w.seed, first_step + i) for i in range(total)])
        else:
            seeds_h = np.stack([S.seed_batch_from_interactions_device(users_d, items_d, w.batch, w.seed, first_step + i)
                                for i in range(total)])
        del users_d, items_d
        torch.cuda.empty_cache()
        X = S.normal_features_device(w.n_nodes, w.dim, w.seed, dt, dev)
    else:
        seeds_h = make_batches(w, inter, args.seeds, first_step, total)
        X = torch.from_numpy(X_h).to(dev, dt)
    Ws = [torch.from_numpy(W).to(dev, dt) for W in Ws_h]
    torch.cuda.synchronize()
    setup_s = time.perf_counter() - t_setup
    seeds_pin = torch.from_numpy(seeds_h).pin_memory()
    seeds_dev = seeds_pin.to(dev)
    dH_h = upstream_grad(w, w.batch)
    dH_pin = torch.from_numpy(dH_h).to(dt).pin_memory()
    dH = dH_pin.to(dev)

    # three sets of block buffers, one per stage of the step's pipeline: the hops of batch i + 2 are sampled and the
    # transposed form of batch i + 1 is built while the forward/backward of batch i runs
    NB = 3
    blocks2 = [E.Blocks(w.n_nodes, w.batch, w.fanouts, dev) for _ in range(NB)]
    blocks = blocks2[0]
    L = len(Ws)
    ctx = torch.empty(E.binding.sage_forward_ctx_bytes(blocks, X, Ws), dtype=torch.uint8, device=dev)
    # outputs, the upstream gradient and a snapshot of the block counts exist once per buffer set, so that the copies
    # of one step's results and of the next step's inputs can run beside the step in between
    H_out2 = [torch.zeros(blocks.caps[0][0], w.hidden, dtype=dt, device=dev) for _ in range(NB)]
    H_out = H_out2[0]
    scratch = torch.empty(E.binding.sage_backward_scratch_bytes(blocks, X, Ws), dtype=torch.uint8, device=dev)
    dWs2 = [[torch.zeros(W.shape, dtype=torch.float32, device=dev) for W in Ws] for _ in range(NB)]
    dX2 = [torch.zeros(blocks.caps[L - 1][1], w.dim, dtype=dt, device=dev) for _ in range(NB)]

    seeds_in2 = [torch.empty(w.batch, dtype=torch.int32, device=dev) for _ in range(NB)]
    dH_in2 = [torch.empty_like(dH) for _ in range(NB)]
    counts_snap2 = [torch.zeros(L, 4, dtype=torch.int32, device=dev) for _ in range(NB)]
    count_total = torch.zeros(L, 4, dtype=torch.int64, device=dev)

    def sample_leg(p, defer=False, transpose=True):
        E.sample_khop(indptr, indices, seeds_in2[p], blocks2[p], w.seed, 0, defer_transpose=defer,
                      edge_cum=edge_cum, transpose=transpose)     # step = the scratch's offset

    def transpose_leg(p):
        E.blocks_transpose(blocks2[p])

    if args.multitask:
        # the two-task step of Sec. 4.2 / 4.3.1: the recommendation gradient and the gradient of the SSL reconstruction
        # loss go through the encoder together (two right-hand sides of one backward pass, weight gradients summed),
        # their norms at the shared input feed one GradNorm step of the task weights
        if w.hidden != w.dim:
            raise SystemExit("--multitask needs hidden == dim (the identity decoder compares H with X)")
        f32 = dict(dtype=torch.float32, device=dev)
        mt = dict(dX_ssl=torch.zeros_like(dX2[0]), dH_ssl=torch.zeros_like(H_out), one=torch.ones(1, **f32),
                  wts=torch.ones(2, **f32), L=torch.ones(2, **f32), L0=torch.ones(2, **f32), g=torch.zeros(2, **f32),
                  scratch=torch.empty(E.binding.sage_backward_multi_scratch_bytes(blocks, X, Ws, 2), dtype=torch.uint8, device=dev))

    def compute_leg(p):
        E.sage_forward(blocks2[p], X, Ws, ctx=ctx, H_out=H_out2[p])
        if not args.multitask:
            E.sage_backward(blocks2[p], X, Ws, ctx, dH_in2[p], dWs=dWs2[p], dX_rows=dX2[p], scratch=scratch)
        else:
            n_seeds_dev, n_rows_dev = blocks2[p].counts[0][0:1], blocks2[p].counts[L - 1][1:2]
            E.ssl_loss(H_out2[p], X, seeds_in2[p], n_seeds_dev, mt["one"], loss=mt["L"][0:1], dH=mt["dH_ssl"])
            # both task gradients through the encoder in one pass: two input gradients, summed weight gradients
            E.sage_backward_multi(blocks2[p], X, Ws, ctx, [dH_in2[p], mt["dH_ssl"]], dWs=dWs2[p], dX_rows=[dX2[p], mt["dX_ssl"]],
                                  scratch=mt["scratch"])
            E.gradient_norms([mt["dX_ssl"], dX2[p]], n_rows_dev, out=mt["g"])      # g[0]: SSL task, g[1]: recommendation task
            E.gradnorm_update(mt["wts"], mt["L"], mt["L0"], mt["g"], 1.0, 0.025)
        count_total.add_(blocks2[p].counts)
        counts_snap2[p].copy_(blocks2[p].counts)

    def step_body():
        """Everything of one training step back to back on fixed buffers (used for warm-up and per-kernel timing)."""
        sample_leg(0, defer=True)
        compute_leg(0)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- record the step as CUDA graphs (no host work between the kernels) and replay them.  Graph p holds the
    # forward/backward of the batch in buffer p and, on two more streams, the transposed form of the batch in buffer
    # p + 1 and the hops of the batch after that into buffer p + 2 (indices mod 3).
    # The forward/backward leg decides the step time, so its stream (and the library's helper stream, which takes its
    # caller's priority) runs at high priority: its kernels get SM slots before the short kernels of the other legs.
    side, side2, side3 = torch.cuda.Stream(priority=-1), torch.cuda.Stream(), torch.cuda.Stream()
    for t in dH_in2:
        t.copy_(dH)
    with torch.cuda.stream(side):
        for i in range(Wm):                              # eager warm-up on the capture stream
            seeds_in2[0].copy_(seeds_dev[i])
            E.sampler_set_step(blocks.scratch, first_step + i)
            step_body()
        for p in range(1, NB):                           # the other buffers and streams, once, eagerly
            seeds_in2[p].copy_(seeds_dev[0])
            E.sampler_set_step(blocks2[p].scratch, first_step)
            with torch.cuda.stream(side2):
                side2.wait_stream(side)
                sample_leg(p, transpose=False)
            with torch.cuda.stream(side3):
                side3.wait_stream(side2)
                transpose_leg(p)
            side.wait_stream(side3)
            compute_leg(p)
    side.synchronize()
    graphs, kernels_per_step = [], 0
    for p in range(NB):
        launches_before = E.launch_count()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            side2.wait_stream(side)
            side3.wait_stream(side)
            with torch.cuda.stream(side2):
                sample_leg((p + 2) % NB, transpose=False)
            with torch.cuda.stream(side3):
                transpose_leg((p + 1) % NB)
            compute_leg(p)
            side.wait_stream(side2)
            side.wait_stream(side3)
        graphs.append(g)
        kernels_per_step = E.launch_count() - launches_before + 2   # + the counter update and snapshot (torch kernels)

    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev_a.record(); ev_b.record()
    torch.cuda.synchronize()

    def leg_alone_ms(body, n):
        """One leg of the step in a CUDA graph of its own, replayed n times back to back with nothing beside it."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            body()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g.replay()
        torch.cuda.synchronize()
        a.record()
        for _ in range(n):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    def hops_then_transposition():
        sample_leg(1, transpose=False)
        transpose_leg(1)

    seeds_in2[1].copy_(seeds_dev[Wm])
    n_leg = max(20, min(K, 200))
    legs_ms = dict(forward_backward=leg_alone_ms(lambda: compute_leg(0), n_leg),
                   hops=leg_alone_ms(lambda: sample_leg(1, transpose=False), n_leg),
                   hops_and_transposition=leg_alone_ms(hops_then_transposition, n_leg))

    def run_step(i):
        """One step, eagerly and back to back (sampling, forward, backward of batch i)."""
        seeds_in2[0].copy_(seeds_dev[i], non_blocking=True)
        E.sampler_set_step(blocks.scratch, first_step + i)
        step_body()

    def prime(i, src):
        """What the two replays before step i would have done: batch i sampled and transposed into buffer i % 3,
        the hops of batch i + 1 into the next buffer."""
        for k, tr in ((i, True), (i + 1, False)):
            seeds_in2[k % NB].copy_(src[k], non_blocking=True)
            E.sampler_set_step(blocks2[k % NB].scratch, first_step + k)
            sample_leg(k % NB, transpose=tr)

    def replay_step(i, src):
        """Forward/backward of batch i beside the transposition of batch i + 1 and the hops of batch i + 2."""
        seeds_in2[(i + 2) % NB].copy_(src[i + 2], non_blocking=True)
        E.sampler_set_step(blocks2[(i + 2) % NB].scratch, first_step + i + 2)
        graphs[i % NB].replay()

    def tapped_step(i, which):
        """One eagerly launched step with events around kernel group `which`.  The device is first kept
        busy for ~1 ms so that the whole step is queued before it starts: the events then bracket the
        kernels alone, not the host's launch latency (events recorded inside a graph cannot be timed)."""
        torch.cuda._sleep(2_000_000)
        E.profile_tap(which, ev_a, ev_b)
        run_step(i)
        torch.cuda.synchronize()
        return ev_a.elapsed_time(ev_b)

    n_tap_steps = min(K, 10)
    tap_ms = {which: float(np.mean([tapped_step(Wm + i, which) for i in range(n_tap_steps)])) for which in TAP_NAMES}
    # the dominant kernel among those on the step's own stream; the weight-gradient product (tap 4) runs on the helper
    # stream beside the input-gradient product and the transposed aggregation, and its tap time includes the time it
    # waits for SMs that those kernels hold
    dominant = max((k for k in tap_ms if k <= 5 and k != 4), key=lambda k: tap_ms[k])

    # ---- the timed region: the K-step replay loop, repeated until the region is at least MIN_TIMED_S long.  Every
    # repetition is bracketed by a barrier and a device synchronisation and timed with CUDA events; the reported step
    # time is the median over the repetitions.
    def timed_loop():
        count_total.zero_()
        prime(Wm, seeds_dev)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(K):
            replay_step(Wm + i, seeds_dev)
        e1.record()
        barrier()
        c = count_total.cpu().numpy()
        if c[:, 3].any():
            raise RuntimeError(f"device status bits set during the timed region: {c[:, 3]}")
        return e0.elapsed_time(e1), c

    probe_ms, _ = timed_loop()                          # untimed repetition: sizes the number of repetitions
    repeats = max(1, min(2000, math.ceil(MIN_TIMED_S * 1e3 / max(probe_ms, 1e-3))))
    clocks = ClockSampler(local)
    clocks.start()
    time.sleep(0.3)                                    # the sampler is polling before the region starts
    barrier()
    t_begin = clocks.mark()
    reps = [timed_loop() for _ in range(repeats)]
    clk = clocks.stop(t_begin, clocks.mark())
    rep_ms = [r[0] for r in reps]
    ms = float(statistics.median(rep_ms))              # one repetition of K steps
    counts = reps[0][1]                                 # [L, 4] summed over the K steps (the same batches in every repetition)
    edges_rank = int(counts[:, 2].sum())
    launches = K * (kernels_per_step + 2)               # + seed copy and step-offset kernel per step
    # the dominant kernel again, timed inside eagerly launched steps over the same batches
    count_total.zero_()
    dom_ms = [tapped_step(Wm + i, dominant) for i in range(min(K, 50))]
    outer_counts = count_total.cpu().numpy()[L - 1] / len(dom_ms)
    max_rows = int(np.ceil(1.3 * outer_counts[1])) + 1024

    # ---- end to end: host buffers in, results out, every step.  Three streams: the step itself; the upload of the
    # next step's inputs (seeds of the batch sampled next, upstream gradient) while the step runs; the download of
    # the step's results while the next step runs: the embeddings, the weight gradients, the counts and -- with_dx --
    # the gradient rows of the input features with their node ids (true count, read from the counts first).
    res_pin2 = [[torch.empty(H_out.shape, dtype=dt).pin_memory()] +
                [torch.empty(W.shape, dtype=torch.float32).pin_memory() for W in Ws] for _ in range(NB)]
    cnt_pin2 = [torch.empty(L, 4, dtype=torch.int32).pin_memory() for _ in range(NB)]
    pin_rows = min(blocks.caps[L - 1][1], max_rows)
    dx_pin2 = [torch.empty(pin_rows, w.dim, dtype=dt).pin_memory() for _ in range(NB)]
    id_pin2 = [torch.empty(pin_rows, dtype=torch.int32).pin_memory() for _ in range(NB)]
    h2d = seeds_pin[0].numel() * 4 + dH_pin.numel() * dH_pin.element_size()
    d2h_fixed = sum(t.numel() * t.element_size() for t in res_pin2[0]) + cnt_pin2[0].numel() * 4
    main_s = torch.cuda.current_stream()
    up_s, down_s = torch.cuda.Stream(), torch.cuda.Stream()
    ev = lambda: torch.cuda.Event()
    done_ev, up_ev, out_ev, cnt_ev = ([ev() for _ in range(NB)] for _ in range(4))

    def e2e_run(first, count, with_dx):
        """Steps first .. first + count - 1; returns (edges their results report, dX bytes downloaded, rows cut off)."""
        edges, dx_bytes, cut = 0, 0, 0
        prime(first, seeds_pin)                                     # batches `first`, `first + 1` into their buffers
        with torch.cuda.stream(up_s):
            up_s.wait_stream(main_s)
            seeds_in2[(first + 2) % NB].copy_(seeds_pin[first + 2], non_blocking=True)
            dH_in2[first % NB].copy_(dH_pin, non_blocking=True)
            up_ev[first % NB].record(up_s)

        def collect(j):
            """Downloads of step j (its counts are already on their way) and the host's read of them."""
            nonlocal edges, dx_bytes, cut
            p = j % NB
            cnt_ev[p].synchronize()
            edges += int(cnt_pin2[p][:, 2].sum())
            if with_dx:
                n_src = int(cnt_pin2[p][L - 1, 1])
                rows = min(n_src, pin_rows)
                cut += n_src - rows
                with torch.cuda.stream(down_s):
                    dx_pin2[p][:rows].copy_(dX2[p][:rows], non_blocking=True)
                    id_pin2[p][:rows].copy_(blocks2[p].t[L - 1]["src_nodes"][:rows], non_blocking=True)
                    out_ev[p].record(down_s)
                dx_bytes += rows * (w.dim * dx_pin2[p].element_size() + 4)

        for i in range(first, first + count):
            p, q = i % NB, (i + 1) % NB
            main_s.wait_event(up_ev[p])                              # inputs of step i are on the device
            if i >= first + NB:
                main_s.wait_event(out_ev[p])                         # the results of step i - 3 have left these buffers
            E.sampler_set_step(blocks2[(i + 2) % NB].scratch, first_step + i + 2)
            graphs[p].replay()
            done_ev[p].record(main_s)
            with torch.cuda.stream(up_s):                            # inputs of step i + 1, beside step i
                if i > first:
                    up_s.wait_event(done_ev[(i - 1) % NB])           # step i - 1 no longer reads these buffers
                seeds_in2[p].copy_(seeds_pin[i + 3], non_blocking=True)    # read by step i + 1 (hops of batch i + 3)
                dH_in2[q].copy_(dH_pin, non_blocking=True)
                up_ev[q].record(up_s)
            with torch.cuda.stream(down_s):                          # results of step i, beside step i + 1
                down_s.wait_event(done_ev[p])
                cnt_pin2[p].copy_(counts_snap2[p], non_blocking=True)
                cnt_ev[p].record(down_s)
                res_pin2[p][0].copy_(H_out2[p], non_blocking=True)
                for t, src in zip(res_pin2[p][1:], dWs2[p]):
                    t.copy_(src, non_blocking=True)
                out_ev[p].record(down_s)
            if i > first:                                            # the caller reads the results of step i - 1
                collect(i - 1)
        collect(first + count - 1)
        torch.cuda.synchronize()
        return edges, dx_bytes, cut

    def e2e_timed(with_dx):
        e2e_run(0, min(Wm, 3), with_dx)
        barrier()
        t0 = time.perf_counter()
        edges, dx_bytes, cut = e2e_run(Wm, K, with_dx)
        barrier()
        return time.perf_counter() - t0, edges, dx_bytes, cut

    e2e_s, e2e_edges, dx_bytes, dx_cut = e2e_timed(True)
    e2e_dev_s, e2e_dev_edges, _, _ = e2e_timed(False)

    # ---- joint step (sampled encoder + ranking tower + BCE, forward and backward) on the same graph
    joint = None
    if with_joint and not on_device:
        joint = run_joint(args, w, E, dev, dt, world, rank, first_step, indptr, indices, X, Ws, inter, indptr_h, indices_h,
                          X_h, Ws_h, (side, side2), barrier, want_cpu)

    # ---- reduce over ranks: slowest rank's time, all ranks' edges
    from paper_2511_20564_b200 import replicas
    (ms, e2e_s, e2e_dev_s), (edges_all, e2e_edges_all, e2e_dev_edges_all) = replicas.reduce_measurements(
        [ms, e2e_s, e2e_dev_s], [edges_rank, e2e_edges, e2e_dev_edges], dev)
    if rank != 0:
        return None

    # ---- roofline of the dominant kernel (algorithmic bytes or flops per launch / mean launch time)
    peaks = measured_peaks()
    es = 2 if w.dtype == "bf16" else 4
    r = w.dim * es
    n_dst, n_src, n_edges = float(outer_counts[0]), float(outer_counts[1]), float(outer_counts[2])
    outer_cap_edges = int(blocks.caps[L - 1][2])
    dom_mean_ms = float(np.mean(dom_ms))
    # both aggregation kernels of the outermost block, whichever kernel dominates.  forward, per entry: id + gathered
    # row; per destination: offsets, self id, self row, [self|mean] row out.  backward, per entry: row id + gathered
    # row; per source: offsets + row out; per destination: self row
    alg_fwd = n_edges * (4 + r) + n_dst * (8 + 4 + r + 2 * r)
    alg_bwd = n_edges * (4 + r) + n_src * (8 + r) + n_dst * r
    if dominant in (1, 2):
        alg = alg_fwd if dominant == 1 else alg_bwd
        roof = dict(bound="hbm", achieved=alg / dom_mean_ms / 1e6, peak=peaks["hbm_gbs"], unit="GB/s")
        roof["frac_of_nominal_8tbs"] = roof["achieved"] / NOMINAL_HBM_GBS
    else:                  # dense products of layer 0: 2 * rows * (2 d) * hidden flop each
        alg = 2.0 * n_dst * 2 * w.dim * w.hidden
        peak = peaks["bf16_tflops"] if w.dtype == "bf16" else fp32_alu_peak_tflops(peaks)
        roof = dict(bound="tensor" if w.dtype == "bf16" else "alu", achieved=alg / dom_mean_ms / 1e9, peak=peak,
                    unit="TFLOP/s")
    aggregation = {
        "outer_block": dict(n_dst=n_dst, n_src=n_src, n_edges=n_edges, row_bytes=r),
        "forward": dict(kernel="sage_aggregate_stream_kernel" if w.dim == 256 and w.dtype == "bf16" and outer_cap_edges >= (1 << 20)
                        else "sage_aggregate_kernel", ms=tap_ms[1], algorithmic_bytes=alg_fwd,
                        **hbm_fractions(alg_fwd / tap_ms[1] / 1e6, peaks)),
        "backward": dict(kernel="seg_run_block_kernel", ms=tap_ms[2], algorithmic_bytes=alg_bwd,
                         **hbm_fractions(alg_bwd / tap_ms[2] / 1e6, peaks))}
    # DRAM bytes per launch: a recorded ncu capture of the same kernel (bytes per entry of the outermost block, taken on
    # this workload or on its reduced-size stand-in) times the entries of one launch here; null without a fresh record
    traffic, traffic_from = None, None
    if dominant in (1, 2) and args.seeds == "activity" and args.beta is None:
        rec = recorded_traffic(f"{w.name}:{'forward' if dominant == 1 else 'backward'}")
        if rec:
            traffic = rec["dram_bytes_per_entry"] * n_edges
            traffic_from = rec.get("captured_on")
    roof.update(frac=roof["achieved"] / roof["peak"], traffic=traffic, traffic_from=traffic_from, kernel=TAP_NAMES[dominant],
                ms_per_launch=dom_mean_ms, algorithmic_units_per_launch=alg, peak_source=peaks["source"])

    d2h_dx = dx_bytes / K
    line = dict(metric=METRIC, value=edges_all / (ms / 1e3), unit=UNIT, n_gpus=world, steps=K, warmup=Wm,
                ms_per_step=ms / K, higher_is_better=True, scaling="weak", vs_baseline=None, dtype=w.dtype,
                data="synthetic",
                timing=dict(repeats=repeats, timed_region_s=sum(rep_ms) / 1e3, ms_per_step_min=min(rep_ms) / K,
                            ms_per_step_max=max(rep_ms) / K, statistic="median over the repetitions of the K-step loop"),
                config=dict(workload=w.name, nodes=w.n_nodes, csr_entries=int(indices.numel()), dim=w.dim, hidden=w.hidden,
                            layers=L, fanouts=list(w.fanouts), batch=w.batch, seeds=args.seeds,
                            sampling="uniform" if args.beta is None else f"weighted, beta={args.beta}",
                            tasks="recommendation gradient + SSL reconstruction loss as two right-hand sides of one backward pass, "
                                  "gradient norms, GradNorm step"
                                  if args.multitask else "recommendation gradient",
                            parallelism=f"replicas x{world}",
                            launch="one CUDA graph replay per step, three streams: forward/backward of batch i beside the "
                                   "transposed form of batch i+1 and the hops of batch i+2 (three sets of block buffers)",
                            l2="inputs larger than L2: feature table + graph = %.0f MB, a new batch every step"
                               % ((X.numel() * es + indices.numel() * 4 + indptr.numel() * 8) / 1e6),
                            edges_per_step=edges_rank / K, setup_s=round(setup_s, 1),
                            generated="on the device (torch)" if on_device else "on the host (numpy)"),
                clocks=clk,
                e2e=dict(value=e2e_edges_all / e2e_s, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h_fixed + d2h_dx,
                         ms_per_step=e2e_s / K * 1e3,
                         results="embeddings, weight gradients, counts, and the feature-gradient rows with their node ids "
                                 "(true count per step)", dx_rows_not_copied=int(dx_cut)),
                e2e_dx_on_device=dict(value=e2e_dev_edges_all / e2e_dev_s, unit=UNIT, h2d_bytes_per_step=h2d,
                                      d2h_bytes_per_step=d2h_fixed, ms_per_step=e2e_dev_s / K * 1e3,
                                      dx_left_on_device_bytes=d2h_dx,
                                      note="same steps with the feature-gradient rows left on the device, where the feature "
                                           "table lives and a sparse update would consume them"),
                gpu_launches=int(launches * repeats),
                roofline=roof, aggregation=aggregation,
                kernel_ms={TAP_NAMES[k].split(" (")[0]: v for k, v in tap_ms.items()},
                legs_alone_ms=dict(legs_ms, note="each leg of the step replayed alone in a CUDA graph of its own (one batch, "
                                                 "nothing beside it); in the step the three legs run side by side"))
    if joint is not None:
        line["joint"] = joint

    if want_cpu:
        import oracle
        oracle.build()
        sample = args.ref_seeds
        dH64 = dH_h[:sample].astype(np.float64)
        note = ""
        X_src = X_h
        if on_device:
            # the oracle samples on a host copy of the device-built CSR and reads the feature rows it needs from the
            # device table (float64 copies of the whole table would not fit the host)
            import psutil
            need = indices.numel() * 4 + indptr.numel() * 8
            if psutil.virtual_memory().available < need * 1.5:
                want_cpu = False
                line["cpu_baseline"] = dict(value=None, unit=UNIT, cores=0, kind="oracle",
                                            sample=f"skipped: the host copy of the graph ({need / 1e9:.1f} GB) does not fit")
            else:
                indptr_h, indices_h = indptr.cpu().numpy(), indices.cpu().numpy()
                X_src = lambda ids: X[torch.from_numpy(np.ascontiguousarray(ids)).to(dev).long()].float().cpu().numpy()
                note = "; graph = host copy of the device-built CSR, feature rows fetched from the device table"
    if want_cpu:
        cum_h = None
        if q_h is not None:
            import oracle
            cum_h = oracle.edge_cumulate(indptr_h, q_h)
        line["cpu_baseline"] = time_oracle(
            lambda n: oracle_step(w, indptr_h, indices_h, X_src, Ws_h, seeds_h[Wm + n][:sample], Wm + n, dH64, cum_h),
            args.cpu_seconds, K, UNIT,
            lambda n, s: f"{n} step(s) on the first {sample} of the {w.batch} seeds of the batch, full "
                         f"sample+forward+backward, {s:.1f} s{note}")
    return line


# ------------------------------------------------------------------------------------------ joint step
def run_joint(args, w, E, dev, dt, world, rank, first_step, indptr, indices, X, Ws, inter, indptr_h, indices_h, X_h, Ws_h,
              streams, barrier, want_cpu):
    """Joint step (sampled encoder + ranking tower + BCE, forward and full backward) on the graph of workload w:
    4 096 training pairs drawn from the interaction list, 64 dense features per pair, tower 512-256-1."""
    import torch
    side, side2 = streams
    K, Wm = args.steps, args.warmup
    P, dd = w.batch, 64
    n_j = min(K, 200)
    jr = np.random.default_rng(4 + rank)
    picks = jr.integers(0, inter[0].size, (n_j + Wm + 1, P))
    pu_h, pi_h = inter[0][picks].astype(np.int32), inter[1][picks].astype(np.int32)
    pu_all, pi_all = torch.from_numpy(pu_h).to(dev), torch.from_numpy(pi_h).to(dev)
    dense_h = jr.standard_normal((P, dd)).astype(np.float32)
    labels_h = S.bernoulli_labels(P, 0.1, 4)
    dense, labels = torch.from_numpy(dense_h).to(dev), torch.from_numpy(labels_h).to(dev)
    zdim = 2 * w.hidden + dd
    Wt_h = [S.glorot_uniform(512, zdim, 4, 40), S.glorot_uniform(256, 512, 4, 41), S.glorot_uniform(1, 256, 4, 42)]
    if w.dtype == "bf16":
        Wt_h = [S.to_bf16_values(a) for a in Wt_h]
    Wt = [torch.from_numpy(a).to(dev, dt) for a in Wt_h]
    bt = [torch.zeros(a.shape[0], dtype=torch.float32, device=dev) for a in Wt_h]
    gate_kw = {}
    if args.gate:
        Wg_h = S.glorot_uniform(zdim, zdim, 4, 43)
        gate_kw = dict(W_gate=torch.from_numpy(Wg_h).to(dev, dt), b_gate=torch.zeros(zdim, dtype=torch.float32, device=dev))
    # two workspaces: the pairs of the next step are turned into seeds and sampled (phase 1) on a second stream
    # while the rest of the current step (phase 2) runs
    js2 = [E.JointStep(indptr, indices, X, P, dd, w.fanouts, Ws, Wt, bt, **gate_kw) for _ in range(2)]
    pu_in2 = [torch.empty_like(pu_all[0]) for _ in range(2)]
    pi_in2 = [torch.empty_like(pi_all[0]) for _ in range(2)]

    def j_sample(p):
        js2[p].run(pu_in2[p], pi_in2[p], dense, labels, 4, 0, phase=1)

    def j_compute(p):
        js2[p].run(pu_in2[p], pi_in2[p], dense, labels, 4, 0, phase=2)

    with torch.cuda.stream(side):
        for i in range(Wm):
            for p in range(2):
                pu_in2[p].copy_(pu_all[i]); pi_in2[p].copy_(pi_all[i])
                E.sampler_set_step(js2[p].ws, first_step + i)
                with torch.cuda.stream(side2):
                    side2.wait_stream(side)
                    j_sample(p)
                side.wait_stream(side2)
                j_compute(p)
    side.synchronize()
    jgraphs, per_step = [], 0
    for p in range(2):
        l0 = E.launch_count()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            side2.wait_stream(side)
            with torch.cuda.stream(side2):
                j_sample(1 - p)
            j_compute(p)
            side.wait_stream(side2)
        jgraphs.append(g)
        per_step = E.launch_count() - l0

    def joint_loop():
        # batch Wm sampled ahead, as the previous replay would have done
        pu_in2[Wm & 1].copy_(pu_all[Wm]); pi_in2[Wm & 1].copy_(pi_all[Wm])
        E.sampler_set_step(js2[Wm & 1].ws, first_step + Wm)
        j_sample(Wm & 1)
        barrier()
        j0, j1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        j0.record()
        for i in range(Wm, Wm + n_j):
            q = (i + 1) & 1
            pu_in2[q].copy_(pu_all[i + 1], non_blocking=True)
            pi_in2[q].copy_(pi_all[i + 1], non_blocking=True)
            E.sampler_set_step(js2[q].ws, first_step + i + 1)
            jgraphs[i & 1].replay()
        j1.record()
        barrier()
        for js in js2:
            if js.n_rows.tolist()[1]:
                raise RuntimeError(f"joint step: device status bits {js.n_rows.tolist()[1]}")
        return j0.elapsed_time(j1)

    probe = joint_loop()
    repeats = max(1, min(2000, math.ceil(MIN_TIMED_S * 1e3 / max(probe, 1e-3))))
    clocks = ClockSampler(dev.index or 0)
    clocks.start()
    time.sleep(0.3)
    t_begin = clocks.mark()
    rep_ms = [joint_loop() for _ in range(repeats)]
    clk = clocks.stop(t_begin, clocks.mark())
    jms = float(statistics.median(rep_ms))
    js = js2[(Wm + n_j - 1) & 1]

    # roofline of the step's widest aggregation kernel group: the transposed aggregation of the outermost block, timed
    # with events around it inside eagerly launched whole steps
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev_a.record(); ev_b.record()                        # the tap wants events whose CUDA handles exist
    torch.cuda.synchronize()
    tap, cnts = [], []
    for i in range(min(n_j, 20)):
        pu_in2[0].copy_(pu_all[Wm + i]); pi_in2[0].copy_(pi_all[Wm + i])
        E.sampler_set_step(js2[0].ws, first_step + Wm + i)
        torch.cuda._sleep(2_000_000)
        E.profile_tap(2, ev_a, ev_b)
        js2[0].run(pu_in2[0], pi_in2[0], dense, labels, 4, 0)
        torch.cuda.synchronize()
        tap.append(ev_a.elapsed_time(ev_b))
        cnts.append(js2[0].activations()["counts"][len(w.fanouts) - 1].tolist())
    peaks = measured_peaks()
    r = w.dim * (2 if w.dtype == "bf16" else 4)
    n_dst, n_src, n_edges = (float(np.mean([c[k] for c in cnts])) for k in range(3))
    alg_bwd = n_edges * (4 + r) + n_src * (8 + r) + n_dst * r
    tms = float(np.mean(tap))
    roof = dict(bound="hbm", achieved=alg_bwd / tms / 1e6, peak=peaks["hbm_gbs"], unit="GB/s", traffic=None,
                kernel=TAP_NAMES[2], ms_per_launch=tms, algorithmic_units_per_launch=alg_bwd, peak_source=peaks["source"],
                outer_block=dict(n_dst=n_dst, n_src=n_src, n_edges=n_edges, row_bytes=r))
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["frac_of_nominal_8tbs"] = roof["achieved"] / NOMINAL_HBM_GBS
    joint = dict(metric="joint_step_samples_per_sec", value=n_j * P * world / (jms / 1e3), unit="pairs/s",
                 ms_per_step=jms / n_j, steps=n_j, pairs_per_step=P, tower="320-512-256-1", dense_dim=dd,
                 gate_fusion=bool(args.gate), loss=float(js.loss), clocks=clk,
                 timing=dict(repeats=repeats, timed_region_s=sum(rep_ms) / 1e3, ms_per_step_min=min(rep_ms) / n_j,
                             ms_per_step_max=max(rep_ms) / n_j, statistic="median over the repetitions of the loop"),
                 gpu_launches=int(per_step * n_j * repeats), roofline=roof,
                 launch="one CUDA graph replay per step: e2egrec_joint_step_phase COMPUTE of the batch beside SAMPLE of the next")
    if want_cpu and indptr_h is not None and not args.gate:
        import oracle
        oracle.build()
        sample = max(32, args.ref_seeds // 2)             # pairs per oracle step (two endpoints each)
        bf16 = w.dtype == "bf16"
        joint["cpu_baseline"] = time_oracle(
            lambda n: (oracle.joint_step(indptr_h, indices_h, X_h, pu_h[Wm + n][:sample], pi_h[Wm + n][:sample],
                                         dense_h[:sample], labels_h[:sample], w.fanouts, Ws_h, Wt_h, None, 4, Wm + n,
                                         bf16=bf16) and sample),
            args.cpu_seconds, n_j, "pairs/s",
            lambda n, s: f"{n} step(s) on the first {sample} of the {P} pairs of the batch, whole joint step, {s:.1f} s")
    return joint


# ------------------------------------------------------------------------------------------ LightGCN on sampled blocks
def run_lightgcn(args, w):
    """Sampling + LightGCN propagation (Eqs. 4-7) on the sampled blocks + its adjoint, per step; same schedule as the
    GraphSAGE step (the sampling of the next batch beside the propagation of the current one)."""
    import torch
    import paper_2511_20564_b200 as E
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    E.lib()
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    users, items = S.bipartite_interactions(w.n_users, w.n_items, w.n_interactions, w.alpha_user, w.alpha_item, w.seed, w.q)
    row_d = torch.cat([torch.from_numpy(users), torch.from_numpy(items)]).to(dev)
    col_d = torch.cat([torch.from_numpy(items), torch.from_numpy(users)]).to(dev)
    indptr, indices, st = E.graph_from_coo(w.n_nodes, row_d, col_d)
    indices = indices.contiguous()
    if int(st):
        raise RuntimeError("graph ingest: node id out of range")
    del row_d, col_d
    deg_h = np.bincount(np.concatenate([users, items]), minlength=w.n_nodes)
    s_h = np.where(deg_h > 0, 1.0 / np.sqrt(np.maximum(deg_h, 1)), 0.0).astype(np.float32)
    s_d = torch.from_numpy(s_h).to(dev)
    X_h = S.normal_features(w.n_nodes, w.dim, w.seed)
    if w.dtype == "bf16":
        X_h = S.to_bf16_values(X_h)
    X = torch.from_numpy(X_h).to(dev, dt)
    K, Wm = args.steps, args.warmup
    seeds_h = make_batches(w, (users, items), args.seeds, 0, K + Wm + 3)
    seeds_dev = torch.from_numpy(seeds_h).to(dev)
    dY_h = upstream_grad(w, w.batch)[:, : w.dim] if w.hidden >= w.dim else np.zeros((w.batch, w.dim), np.float32)
    NB = 3                                               # hops of batch i+2, transposed form of batch i+1, compute of batch i
    blocks2 = [E.Blocks(w.n_nodes, w.batch, w.fanouts, dev) for _ in range(NB)]
    seeds_in2 = [torch.empty(w.batch, dtype=torch.int32, device=dev) for _ in range(NB)]
    Y = torch.zeros(blocks2[0].caps[0][0], w.dim, dtype=dt, device=dev)
    dY = torch.zeros_like(Y)
    dY[: w.batch] = torch.from_numpy(dY_h).to(dev, dt)
    dX = torch.zeros(blocks2[0].caps[-1][1], w.dim, dtype=dt, device=dev)
    _, ctx = E.lightgcn_sampled_forward(blocks2[0], X, s_d, Y=Y)
    _, scratch = E.lightgcn_sampled_backward(blocks2[0], ctx, dY, dX_rows=dX)
    count_total = torch.zeros(len(w.fanouts), 4, dtype=torch.int64, device=dev)

    def sample_leg(p, transpose=True):
        E.sample_khop(indptr, indices, seeds_in2[p], blocks2[p], w.seed, 0, transpose=transpose)

    def compute_leg(p):
        E.lightgcn_sampled_forward(blocks2[p], X, s_d, ctx=ctx, Y=Y)
        E.lightgcn_sampled_backward(blocks2[p], ctx, dY, dX_rows=dX, scratch=scratch)
        count_total.add_(blocks2[p].counts)

    # the same three-stage pipeline as the GraphSAGE step; here the two sampling legs are the longer ones and run at
    # high priority: their short dependent kernels take the next free slots of an SM
    side, side2, side3 = torch.cuda.Stream(), torch.cuda.Stream(priority=-1), torch.cuda.Stream(priority=-1)
    with torch.cuda.stream(side):
        for i in range(max(Wm, 3)):
            for p in range(NB):
                seeds_in2[p].copy_(seeds_dev[i])
                E.sampler_set_step(blocks2[p].scratch, i)
                with torch.cuda.stream(side2):
                    side2.wait_stream(side)
                    sample_leg(p, transpose=False)
                with torch.cuda.stream(side3):
                    side3.wait_stream(side2)
                    E.blocks_transpose(blocks2[p])
                side.wait_stream(side3)
                compute_leg(p)
    side.synchronize()
    graphs = []
    l0 = E.launch_count()
    for p in range(NB):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            side2.wait_stream(side)
            side3.wait_stream(side)
            with torch.cuda.stream(side2):
                sample_leg((p + 2) % NB, transpose=False)
            with torch.cuda.stream(side3):
                E.blocks_transpose(blocks2[(p + 1) % NB])
            compute_leg(p)
            side.wait_stream(side2)
            side.wait_stream(side3)
        graphs.append(g)
    kernels_per_step = (E.launch_count() - l0) // NB + 1

    def prime(i):
        for k, tr in ((i, True), (i + 1, False)):
            seeds_in2[k % NB].copy_(seeds_dev[k], non_blocking=True)
            E.sampler_set_step(blocks2[k % NB].scratch, k)
            sample_leg(k % NB, transpose=tr)

    def replay_step(i):
        seeds_in2[(i + 2) % NB].copy_(seeds_dev[i + 2], non_blocking=True)
        E.sampler_set_step(blocks2[(i + 2) % NB].scratch, i + 2)
        graphs[i % NB].replay()

    def timed_loop():
        prime(Wm)
        count_total.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(K):
            replay_step(Wm + i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    probe = timed_loop()
    repeats = max(1, min(2000, math.ceil(MIN_TIMED_S * 1e3 / max(probe, 1e-3))))
    clocks = ClockSampler(0)
    clocks.start()
    time.sleep(0.3)
    t_begin = clocks.mark()
    rep_ms = [timed_loop() for _ in range(repeats)]
    clk = clocks.stop(t_begin, clocks.mark())
    ms = float(statistics.median(rep_ms))
    counts = count_total.cpu().numpy()
    if counts[:, 3].any():
        raise RuntimeError(f"device status bits set during the timed region: {counts[:, 3]}")
    edges = int(counts[:, 2].sum())
    line = dict(metric="sampled_lightgcn_sample_fwd_bwd_edges_per_sec", value=edges / (ms / 1e3), unit=UNIT, n_gpus=1, steps=K,
                warmup=Wm, ms_per_step=ms / K, higher_is_better=True, scaling="weak", vs_baseline=None, dtype=w.dtype,
                data="synthetic",
                timing=dict(repeats=repeats, timed_region_s=sum(rep_ms) / 1e3, statistic="median over the repetitions"),
                config=dict(workload=w.name, backbone="lightgcn", nodes=w.n_nodes, csr_entries=int(indices.numel()), dim=w.dim,
                            layers=len(w.fanouts), fanouts=list(w.fanouts), batch=w.batch, seeds=args.seeds,
                            launch="one CUDA graph replay per step, three streams: propagation and adjoint of batch i beside "
                                   "the transposed form of batch i+1 and the hops of batch i+2", edges_per_step=edges / K),
                clocks=clk, gpu_launches=int(K * (kernels_per_step + 2) * repeats))
    if not args.no_cpu_baseline:
        import oracle
        oracle.build()
        row, col = S.undirected_coo(users, items)
        indptr_h, indices_h = S.coo_to_csr(w.n_nodes, row, col)
        sample = args.ref_seeds

        def ostep(n):
            blocks = oracle.sample_khop(indptr_h, indices_h, seeds_h[Wm + n][:sample], w.fanouts, w.seed, Wm + n)
            _, octx = oracle.lightgcn_sampled_forward(blocks, X_h, s_h, w.dtype == "bf16")
            oracle.lightgcn_sampled_backward(blocks, octx, dY_h[:sample], w.dtype == "bf16")
            return sum(b["n_edges"] for b in blocks)

        line["cpu_baseline"] = time_oracle(ostep, args.cpu_seconds, K, UNIT,
                                           lambda n, s: f"{n} step(s) on the first {sample} of the {w.batch} seeds of the batch, {s:.1f} s")
    return line


# ------------------------------------------------------------------------------------------ whole-graph aggregation
def run_fullgraph(args):
    """Mean aggregation over the whole graph (no sampling) and its transpose: one forward (CSR gather) and one
    backward (CSC gather) per step, on a directed power-law graph."""
    import torch
    import paper_2511_20564_b200 as E
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n = int(5_000_000 * args.scale)
    m = int(100_000_000 * args.scale)
    d = 64
    t0 = time.perf_counter()
    dst, src = S.powerlaw_directed(n, m, 1.1, 2)
    indptr, indices, st1 = E.graph_from_coo(n, torch.from_numpy(dst).to(dev), torch.from_numpy(src).to(dev))
    indices = indices.contiguous()
    csc_ptr, csc_row, _, st2 = E.csr_transpose(indptr, indices, n)
    csc_row = csc_row.contiguous()
    if int(st1) or int(st2):
        raise RuntimeError("graph ingest: node id out of range")
    deg_d = (indptr[1:] - indptr[:-1])
    inv_deg = torch.where(deg_d > 0, 1.0 / deg_d.clamp(min=1).float(), torch.zeros((), device=dev)).float()
    max_degree = int(deg_d.max())
    torch.cuda.synchronize()
    setup_s = time.perf_counter() - t0
    X_h = S.to_bf16_values(S.normal_features(n, d, 2))
    G_h = S.to_bf16_values(S.normal_features(n, d, 2, stream=11))
    cu = lambda a: torch.from_numpy(a).to(dev)
    X, G = cu(X_h).to(torch.bfloat16), cu(G_h).to(torch.bfloat16)
    out = torch.empty(n, d, dtype=torch.bfloat16, device=dev)
    dX = torch.empty(n, d, dtype=torch.bfloat16, device=dev)
    _, ws_f = E.aggregate_forward(indptr, indices, X, out)
    _, ws_b = E.aggregate_backward(csc_ptr, csc_row, inv_deg, G, dX)
    Wm = max(args.warmup, 3)

    def fwd():
        E.aggregate_forward(indptr, indices, X, out, ws_f)

    def bwd():
        E.aggregate_backward(csc_ptr, csc_row, inv_deg, G, dX, ws_b)

    for _ in range(Wm):
        fwd(); bwd()
    torch.cuda.synchronize()
    pa, pb, pc = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    pa.record(); fwd(); pb.record(); bwd(); pc.record()
    torch.cuda.synchronize()
    # as many steps as the caller asked for, and at least enough for a timed region of MIN_TIMED_S
    K = max(args.steps, math.ceil(MIN_TIMED_S * 1e3 / max(pa.elapsed_time(pc), 1e-3)))
    clocks = ClockSampler(0)
    clocks.start()
    time.sleep(0.3)
    t_begin = clocks.mark()
    l0 = E.launch_count()
    ef = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(K)]
    for a, b, c in ef:
        a.record(); fwd(); b.record(); bwd(); c.record()
    torch.cuda.synchronize()
    clk = clocks.stop(t_begin, clocks.mark())
    launches = E.launch_count() - l0
    t_f = float(statistics.median([a.elapsed_time(b) for a, b, _ in ef]))
    t_b = float(statistics.median([b.elapsed_time(c) for _, b, c in ef]))
    ms = ef[0][0].elapsed_time(ef[-1][2])
    # end to end: features from pinned host memory in, aggregated rows out, every step
    X_pin, G_pin = X.cpu().pin_memory(), G.cpu().pin_memory()
    out_pin, dX_pin = torch.empty_like(X_pin), torch.empty_like(X_pin)
    ke = max(2, min(K, 5))
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(ke):
        X.copy_(X_pin, non_blocking=True); G.copy_(G_pin, non_blocking=True)
        fwd(); bwd()
        out_pin.copy_(out, non_blocking=True); dX_pin.copy_(dX, non_blocking=True)
        torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / ke
    peaks = measured_peaks()
    r = d * 2
    # (no-reuse) per entry: id + gathered row; per row: two offsets + the output row; backward + the per-entry weight 1/deg
    alg_f = m * (4 + r) + n * (16 + r)
    alg_b = m * (4 + 4 + r) + n * (16 + r)
    # (compulsory) every distinct byte once: the table in, the table out, the ids, the offsets (+ the weights)
    comp_f = n * r * 2 + m * 4 + n * 16
    comp_b = comp_f + n * 4

    def direction(name, t_ms, alg, comp):
        rec = recorded_traffic(f"fullgraph:{name}")
        out_d = dict(ms=t_ms, edges_per_s=m / (t_ms / 1e3),
                     no_reuse=dict(bytes=alg, **hbm_fractions(alg / t_ms / 1e6, peaks)),
                     compulsory=dict(bytes=comp, **hbm_fractions(comp / t_ms / 1e6, peaks)),
                     dram_counter=None)
        if rec:   # bytes per entry measured by ncu on the reduced graph named in the record, times this graph's entries
            tr = rec["dram_bytes_per_entry"] * m
            out_d["dram_counter"] = dict(bytes=tr, captured_on=rec.get("captured_on"), **hbm_fractions(tr / t_ms / 1e6, peaks))
        return out_d

    fwd_d, bwd_d = direction("forward", t_f, alg_f, comp_f), direction("backward", t_b, alg_b, comp_b)
    big, big_d = ("fwd", fwd_d) if t_f >= t_b else ("bwd", bwd_d)
    roof = dict(bound="hbm", achieved=big_d["no_reuse"]["gbs"], peak=peaks["hbm_gbs"], unit="GB/s",
                traffic=big_d["dram_counter"]["bytes"] if big_d["dram_counter"] else None,
                kernel=f"seg_run_kernel+seg_final_kernel ({big})", ms_per_launch=big_d["ms"],
                algorithmic_units_per_launch=big_d["no_reuse"]["bytes"], peak_source=peaks["source"],
                frac_of_nominal_8tbs=big_d["no_reuse"]["frac_of_nominal_8tbs"],
                compulsory_frac=big_d["compulsory"]["frac_of_measured_copy"],
                dram_counter_frac=big_d["dram_counter"]["frac_of_measured_copy"] if big_d["dram_counter"] else None,
                note="achieved = algorithmic no-reuse bytes / time; the compulsory-bytes and DRAM-counter fractions beside it")
    roof["frac"] = roof["achieved"] / roof["peak"]
    line = dict(metric="fullgraph_mean_aggregation_fwd_bwd_edges_per_sec", value=m / ((t_f + t_b) / 1e3), unit="edges/s",
                n_gpus=1, steps=K, warmup=Wm, ms_per_step=t_f + t_b, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16", data="synthetic",
                timing=dict(timed_region_s=ms / 1e3, statistic="median over the steps, forward and backward timed apart"),
                config=dict(workload="fullgraph", nodes=n, csr_entries=m, dim=d, alpha=1.1, max_degree=max_degree,
                            l2="inputs larger than L2 (features %.0f MB, indices %.0f MB)" % (n * r / 1e6, m * 4 / 1e6),
                            ingest_s=round(setup_s, 1)),
                forward=fwd_d, backward=bwd_d, clocks=clk,
                e2e=dict(value=m / e2e_s, unit="edges/s", h2d_bytes_per_step=2 * n * r, d2h_bytes_per_step=2 * n * r,
                         ms_per_step=e2e_s * 1e3),
                gpu_launches=int(launches), roofline=roof)
    if not args.no_cpu_baseline:
        import oracle
        oracle.build()
        rows = min(n, 200_000)
        keep = dst < rows                                           # host CSR of the first rows only, for the oracle
        indptr_h, indices_h = S.coo_to_csr(rows, dst[keep], src[keep])
        line["cpu_baseline"] = time_oracle(
            lambda k: (oracle.mean_aggregate(indptr_h, indices_h, X_h, True) is not None) * int(indptr_h[rows]),
            args.cpu_seconds, 3, "edges/s",
            lambda k, s: f"{k} forward mean aggregation(s) of the first {rows} rows ({int(indptr_h[rows])} entries), {s:.1f} s")
    return line


def free_device_memory():
    import torch
    gc.collect()
    torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(S.WORKLOADS) + ["fullgraph"],
                    help="default: `large` with `medium`, the joint step and `fullgraph` as sub-records")
    ap.add_argument("--scale", type=float, default=1.0, help="fullgraph only: fraction of the 5 M node / 100 M entry graph")
    ap.add_argument("--ref-seeds", type=int, default=256, help="seeds per step given to the CPU oracle")
    ap.add_argument("--cpu-seconds", type=float, default=8.0, help="time budget of each CPU-oracle timing (all cores, one core)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-joint", action="store_true", help="skip the joint-step measurement")
    ap.add_argument("--no-sub", action="store_true", help="default run: skip the sub-records")
    ap.add_argument("--gate", action="store_true", help="joint step with the gating fusion of the tower's input (Sec. 4.3.2)")
    ap.add_argument("--backbone", default="sage", choices=["sage", "lightgcn"],
                    help="lightgcn: sampling + LightGCN propagation on the sampled blocks + its adjoint (no weights)")
    ap.add_argument("--multitask", action="store_true",
                    help="add the SSL reconstruction task: second backward pass, gradient norms, GradNorm weight step")
    ap.add_argument("--beta", type=float, default=None,
                    help="weighted neighbour sampling p ~ omega^beta with synthetic log-normal omega (default: uniform)")
    ap.add_argument("--seeds", default="activity", choices=["activity", "uniform"],
                    help="how seed batches are drawn (see make_batches)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    suite = args.workload is None
    name = "large" if suite else args.workload

    if args.impl == "reference":
        if name == "fullgraph":
            raise SystemExit("--impl reference runs the sampled workloads")
        line = run_reference(args, S.WORKLOADS[name])
        if line is not None:
            print(json.dumps(line), flush=True)
        return
    if name == "fullgraph":
        if rank == 0:
            print(json.dumps(run_fullgraph(args)), flush=True)
        return
    if args.backbone == "lightgcn":
        if rank == 0:
            print(json.dumps(run_lightgcn(args, S.WORKLOADS[name])), flush=True)
        return

    import torch
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        dist.init_process_group("nccl", device_id=torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0"))))
    line = run_ours(args, S.WORKLOADS[name], with_joint=not suite and not args.no_joint)
    if suite and not args.no_sub and world == 1:
        # the other configurations, each with its own roofline, clocks and CPU baseline
        free_device_memory()
        medium = run_ours(args, S.WORKLOADS["medium"], with_joint=not args.no_joint)
        free_device_memory()
        sub = dict(medium=medium)
        if medium is not None and "joint" in medium:
            sub["joint"] = medium.pop("joint")
        sub["fullgraph"] = run_fullgraph(args)
        line["sub"] = sub
    if line is not None:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
