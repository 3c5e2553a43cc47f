#!/usr/bin/env python
"""Benchmark of the int8 inference path of Q8BERT on B200.

One "step" is one pass of the whole hot path over one batch of synthetic BERT-shaped input: the
Int8 embedding gather for the batch's tokens, then for each of the four fully-connected layers of
an encoder block (QKV, attention-out, FFN1 + GELU, FFN2) the activation quantiser (Eq. 1, static
scale from Eq. 4) followed by the tcgen05 Int8 GEMM with its fused bias / dequantise / GELU
epilogue.  Weight quantisation (Eq. 3) and scale calibration (Eq. 4) are one-time set-up and are
not timed.

    python bench.py --gpus 1 --steps K --warmup W            # this library
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, bounded sample

Prints ONE JSON line (rank 0).  `value` is TOPS (2*M*N*K summed over the four GEMMs, divided by the
step time) with inputs resident in HBM; `e2e` is the same metric with host buffers and the
host<->device copies inside the timed region.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1910_06188_b200 import dist_util, synth  # noqa: E402

WORKLOADS = {
    # name: (config index, model dims, description)
    "bert_large_fc": (4, synth.BERT_LARGE, "BERT-Large FC set, batch 64 x seq 384 (M=24576 tokens)"),
    "bert_base_fc": (2, synth.BERT_BASE, "BERT-Base FC set, batch 32 x seq 128 (M=4096 tokens)"),
}
# dram__bytes_read.sum + dram__bytes_write.sum of the tcgen05 GEMM per launch on the BERT-Large FC set, from the
# ncu captures summarised in profiles/gemm_tcgen05_dram_traffic_m24576.md (one layer resident per capture).  Below the
# algorithmic bytes because part of each output is still dirty in the 126 MB L2 when the kernel ends.
GEMM_DRAM_TRAFFIC = {"bert_large_fc": {"qkv": 269605632, "attn_out": 66903040, "ffn1": 371766784, "ffn2": 164554496}}
NOMINAL_INT8_OVER_BF16 = 2.0  # dense tensor peak ratio int8 : bf16 (4.5 : 2.25 POPS nominal)
GEMM_REPS = 4   # launches per event pair in the per-kernel pass
QUANT_REPS = 4  # times each group of equal-sized quantise passes is repeated per event pair
EMB_REPS = 4    # embedding gathers per event pair in the per-kernel pass
EMB_TABLES = 6  # copies of the embedding table the L2-cold gather figure rotates over (6 x 31 MB > L2)
REPLAY_SAMPLES = 100  # individually timed replays of the step for the median / best figures
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def make_layers(cfg_index: int, dims: dict):
    """Host tensors of the four FC layers: activation, calibration batch, weight, bias."""
    M = dims["batch"] * dims["seq"]
    layers = []
    for i, (name, K, N, act) in enumerate(synth.fc_set(dims["hidden"], dims["ffn"])):
        layers.append(dict(
            name=name, M=M, K=K, N=N, act=act,
            X=synth.activation(M, K, synth.seed_for(cfg_index, 10 * i)),
            calib=synth.activation(M, K, synth.seed_for(cfg_index, 10 * i + 1)),
            W=synth.weight(N, K, synth.seed_for(cfg_index, 10 * i + 2)),
            b=synth.bias(N, synth.seed_for(cfg_index, 10 * i + 3)),
        ))
    return M, layers


def total_ops(layers):
    return sum(2.0 * L["M"] * L["N"] * L["K"] for L in layers)


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, v in names.items():
                    if bits & v:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# --------------------------------------------------------------------------- the CPU oracle arm
def run_reference(args):
    """Times the CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import q8_oracle as o  # the one place besides cpu_baseline where bench.py runs the oracle

    cfg_index, dims, desc = WORKLOADS[args.workload]
    M_full = dims["batch"] * dims["seq"]
    rows = M_full if args.reference_rows <= 0 else min(args.reference_rows, M_full)
    layers = []
    for i, (name, K, N, act) in enumerate(synth.fc_set(dims["hidden"], dims["ffn"])):
        X = synth.activation(rows, K, synth.seed_for(cfg_index, 10 * i))
        W = synth.weight(N, K, synth.seed_for(cfg_index, 10 * i + 2))
        b = synth.bias(N, synth.seed_for(cfg_index, 10 * i + 3))
        Wq, S_w, _ = o.quantize_weight(W)
        S_x, _ = o.scale_from_absmax(o.absmax(X))
        layers.append(dict(M=rows, K=K, N=N, act=act, X=X, Wq=Wq, S_w=S_w, S_x=S_x, b=b))
    ops = total_ops(layers)

    def step():
        for L in layers:
            o.linear(L["X"], L["Wq"], L["S_w"], L["S_x"], L["b"], L["act"])

    # One step is the whole workload (all token rows of the four layers), which takes the oracle seconds; the
    # requested warm-up and step counts are cut so that the run stays within --reference-budget-s seconds.
    t0 = time.perf_counter()
    step()
    first = time.perf_counter() - t0
    budget = max(args.reference_budget_s - first, first)
    steps = max(1, min(args.steps, int(budget / first)))
    warm_done = 1
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    value = ops / dt / 1e12
    cores = os.cpu_count()
    sample = f"{rows} of {M_full} token rows of each of the 4 FC layers per step, {steps} timed step(s) after {warm_done} warm-up"
    line = {
        "impl": "reference", "metric": "q8_linear_int8_tops", "value": value, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm_done, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "description": desc, "sample": sample,
                   "steps_requested": args.steps, "warmup_requested": args.warmup,
                   "tokens_per_step": rows},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# --------------------------------------------------------------------------- this library
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_1910_06188_b200 import binding as q8

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    q8.load()

    if args.profile_mode and args.encoder_kernel:
        return profile_encoder_kernel(args, torch, q8)

    cfg_index, dims, desc = WORKLOADS[args.workload]
    # weak scaling: every rank owns one full batch of M tokens (rows are independent given static
    # scales, so there is no data-path collective); rank r draws its batch from its own seeds.
    M, layers = make_layers(dist_util.rank_config(cfg_index, rank), dims)
    if args.layers:
        keep = set(args.layers.split(","))
        layers = [L for L in layers if L["name"] in keep]
    ops = total_ops(layers)
    H, V = dims["hidden"], dims["vocab"]
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()

    # ---- one-time set-up (not timed): Eq. 3 weights, Eq. 4 scales, embedding table
    for L in layers:
        L["Xd"] = torch.from_numpy(L["X"]).to(dev)
        L["bd"] = torch.from_numpy(L["b"]).to(dev)
        L["Wq"], L["S_w"] = q8.q8_quantize_weight(torch.from_numpy(L["W"]).to(dev))
        state = q8.new_calibrate_state(dev)
        q8.q8_calibrate(torch.from_numpy(L["calib"]).to(dev), 0.9999, state)
        L["S_x"] = q8.calibrate_S_x(state).clone()
        L["Y"] = torch.empty((L["M"], L["N"]), dtype=torch.float32, device=dev)
        L["ws"] = q8.new_workspace(L["M"], L["N"], L["K"], dev)
        L["Xq"] = torch.empty((L["M"], L["K"]), dtype=torch.int8, device=dev)
        del L["calib"], L["W"]
    E = synth.embedding_table(V, H, synth.seed_for(cfg_index, 90))
    Eq, S_e = q8.q8_quantize_weight(torch.from_numpy(E).to(dev))
    ids = torch.from_numpy(synth.token_ids(M, V, synth.seed_for(dist_util.rank_config(cfg_index, rank), 91))).to(dev)
    emb_out = torch.empty((M, H), dtype=torch.float32, device=dev)
    torch.cuda.synchronize()

    launches_per_step = 0
    profile_S_y = None
    if args.profile_mode and args.profile_int8_out:
        profile_S_y = torch.full((1,), 20.0, device=dev)
        for L in layers:
            L["Yq_prof"] = torch.empty((L["M"], L["N"]), dtype=torch.int8, device=dev)

    # The four FC layers of the set (and the embedding gather) are independent of one another, so with
    # --streams > 1 each runs on its own stream: the HBM-bound quantise / gather passes of one layer overlap the
    # GEMM of another.  Every step forks from and joins back into the timed stream.
    n_streams = max(1, min(args.streams, 5))
    all_side = [torch.cuda.Stream(device=dev) for _ in range(4)]
    fork, all_joins = torch.cuda.Event(), [torch.cuda.Event() for _ in all_side]

    def step(streams=None):
        nonlocal launches_per_step
        streams = n_streams if streams is None else streams
        side, joins = all_side[:streams - 1], all_joins[:streams - 1]
        n = 0
        work = [lambda: q8.q8_embedding(ids, Eq, S_e, out=emb_out)]
        for L in layers:
            if args.profile_mode and args.profile_int8_out:
                # for ncu captures of the re-quantising epilogue: the layer emits only Int8, at a fixed scale
                work.append(lambda L=L: q8.q8_linear_requant(L["Xd"], L["Wq"], L["S_w"], L["S_x"], L["bd"], L["act"],
                                                             profile_S_y, Yq=L["Yq_prof"], workspace=L["ws"]))
                continue
            work.append(lambda L=L: q8.q8_linear(L["Xd"], L["Wq"], L["S_w"], L["S_x"], L["bd"], L["act"], Y=L["Y"],
                                                 workspace=L["ws"]))
        if not side:
            for w in work:
                w()
                n += q8.q8_last_launch_info()["launches"]
        else:
            # biggest jobs first (FFN2's 503 MB quantise pass, then FFN1), round-robin over main + side streams
            order = sorted(range(len(work)), key=lambda i: -(layers[i - 1]["M"] * layers[i - 1]["K"] if i else 0))
            fork.record(stream)
            lanes = [stream] + side
            for s_ in side:
                s_.wait_event(fork)
            for j, i in enumerate(order):
                with torch.cuda.stream(lanes[j % len(lanes)]):
                    work[i]()
                    n += q8.q8_last_launch_info()["launches"]
            for s_, ev in zip(side, joins):
                ev.record(s_)
                stream.wait_event(ev)
        launches_per_step = n

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    for L in layers:
        code, bits = q8.q8_poll_status(L["ws"])
        if code != q8.Q8_OK:
            raise SystemExit(f"device status {code} ({q8.status_string(code)}) on layer {L['name']}")

    # One step is a fixed sequence of launches on fixed buffers, so it is captured once in a CUDA graph and the
    # timed region replays that graph (no host work between the kernels); --no-graph times the eager launches.
    step_graph = None
    if not args.no_graph and not args.profile_mode and n_streams == 1:
        try:
            step_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(step_graph, capture_error_mode="thread_local"):
                step()
            for _ in range(3):
                step_graph.replay()
            barrier()
        except Exception as ex:  # capture is an optimisation of the launch path only
            print(f"[bench] CUDA graph capture failed ({ex}); timing eager launches", file=sys.stderr)
            step_graph = None
            step()
            barrier()

    # ---- timed region: K whole steps, device time, max over ranks
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    eager_ms = None
    with sampler:
        barrier()
        ev0.record(stream)
        for _ in range(args.steps):
            if step_graph is not None:
                step_graph.replay()
            else:
                step()
        ev1.record(stream)
        barrier()
        ms = ev0.elapsed_time(ev1)
        # the same step, each repetition between its own pair of events (no host synchronisation in between):
        # median and best of REPLAY_SAMPLES beside the mean of the K-step region
        per_step_ms = []
        if not args.profile_mode:
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(REPLAY_SAMPLES + 1)]
            marks[0].record(stream)
            for i in range(REPLAY_SAMPLES):
                if step_graph is not None:
                    step_graph.replay()
                else:
                    step()
                marks[i + 1].record(stream)
            barrier()
            per_step_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(REPLAY_SAMPLES)]
        if step_graph is not None:
            # the same K steps launched eagerly from the host, reported beside the graph-replayed figure
            ev0.record(stream)
            for _ in range(args.steps):
                step()
            ev1.record(stream)
            barrier()
            eager_ms = ev0.elapsed_time(ev1) / args.steps

        # ---- per-kernel pass (same launches, events around each kernel): roofline of the dominant kernel
        nl = len(layers)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(nl)]
        t_quant, t_gemm = [0.0] * nl, [0.0] * nl
        # FFN1 handing its GELU output to FFN2 as Int8 only (Eq. 1 at FFN2's Eq. 4 scale, fused into the epilogue)
        i8 = next((i for i, L in enumerate(layers) if L["name"] == "ffn1"), None)
        i8_consumer = next((L for L in layers if L["name"] == "ffn2"), None)
        t_i8 = 0.0
        ev_i0, ev_i1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev_c0, ev_c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_emb_cold = 0.0
        ev_e0, ev_e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_emb = 0.0
        ksteps = 0 if args.profile_mode else min(args.steps, 50)
        # quantise passes of equal size are timed as one back-to-back group (distinct inputs, together larger than
        # L2), so that the event overhead is shared; the group's time is split evenly among its members
        groups = {}
        for i, L in enumerate(layers):
            groups.setdefault(L["M"] * L["K"], []).append(i)
        gev = {k: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for k in groups}
        # The launches between two events are replayed from a CUDA graph, so the events see device time without
        # host gaps: each layer's GEMM_REPS back-to-back GEMM launches, each group of quantise passes, and
        # EMB_REPS embedding gathers that alternate between two output buffers (together larger than L2).
        gemm_graphs, quant_graphs, emb_graph, i8_graph, emb_cold_graph = [], {}, None, None, None
        emb_out2 = torch.empty_like(emb_out) if ksteps > 0 else None
        Yq_i8 = None
        if ksteps > 0 and i8 is not None and i8_consumer is not None:
            Yq_i8 = torch.empty((layers[i8]["M"], layers[i8]["N"]), dtype=torch.int8, device=dev)
        else:
            i8 = None
        # L2-cold gather: the tokens of the batch look their rows up in EMB_TABLES copies of the table in turn
        Eq_copies = [Eq] + [Eq.clone() for _ in range(EMB_TABLES - 1)] if ksteps > 0 else []

        def run_i8():
            L = layers[i8]
            for _ in range(GEMM_REPS):
                q8.q8_linear_q_requant(L["Xq"], L["S_x"], L["Wq"], L["S_w"], L["bd"], L["act"], i8_consumer["S_x"], Yq=Yq_i8)

        def run_emb_cold():
            for r in range(EMB_TABLES):
                q8.q8_embedding(ids, Eq_copies[r], S_e, out=emb_out if r % 2 == 0 else emb_out2)
        if not args.no_graph and ksteps > 0:
            try:
                for L in layers:
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, capture_error_mode="thread_local"):
                        for _ in range(GEMM_REPS):
                            q8.q8_linear_q(L["Xq"], L["S_x"], L["Wq"], L["S_w"], L["bd"], L["act"], Y=L["Y"])
                    gemm_graphs.append(g)
                for k, members in groups.items():
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, capture_error_mode="thread_local"):
                        for _ in range(QUANT_REPS):
                            for i in members:
                                q8.q8_quantize_activation(layers[i]["Xd"], layers[i]["S_x"], Xq=layers[i]["Xq"])
                    quant_graphs[k] = g
                if i8 is not None:
                    run_i8()
                    i8_graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(i8_graph, capture_error_mode="thread_local"):
                        run_i8()
                run_emb_cold()
                emb_cold_graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(emb_cold_graph, capture_error_mode="thread_local"):
                    run_emb_cold()
                emb_graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(emb_graph, capture_error_mode="thread_local"):
                    for r in range(EMB_REPS):
                        q8.q8_embedding(ids, Eq, S_e, out=emb_out if r % 2 == 0 else emb_out2)
                torch.cuda.synchronize()
            except Exception as ex:
                print(f"[bench] CUDA graph capture of the per-kernel pass failed ({ex}); timing eager launches", file=sys.stderr)
                gemm_graphs, quant_graphs, emb_graph, i8_graph, emb_cold_graph = [], {}, None, None, None
        for _ in range(ksteps):
            # the GEMMs first (right after the synchronisation below, i.e. from the same state as in a step), then the
            # HBM-bound passes
            for i, L in enumerate(layers):
                evs[i][1].record(stream)
                if gemm_graphs:
                    gemm_graphs[i].replay()
                else:
                    for _ in range(GEMM_REPS):  # back to back, so that the event overhead is shared by several launches
                        q8.q8_linear_q(L["Xq"], L["S_x"], L["Wq"], L["S_w"], L["bd"], L["act"], Y=L["Y"])
                evs[i][2].record(stream)
            if i8 is not None:
                ev_i0.record(stream)
                if i8_graph is not None:
                    i8_graph.replay()
                else:
                    run_i8()
                ev_i1.record(stream)
            for k, members in groups.items():
                gev[k][0].record(stream)
                if k in quant_graphs:
                    quant_graphs[k].replay()
                else:
                    for _ in range(QUANT_REPS):
                        for i in members:
                            q8.q8_quantize_activation(layers[i]["Xd"], layers[i]["S_x"], Xq=layers[i]["Xq"])
                gev[k][1].record(stream)
            ev_e0.record(stream)
            if emb_graph is not None:
                emb_graph.replay()
            else:
                for r in range(EMB_REPS):
                    q8.q8_embedding(ids, Eq, S_e, out=emb_out if r % 2 == 0 else emb_out2)
            ev_e1.record(stream)
            ev_c0.record(stream)
            if emb_cold_graph is not None:
                emb_cold_graph.replay()
            else:
                run_emb_cold()
            ev_c1.record(stream)
            torch.cuda.synchronize()
            t_emb += ev_e0.elapsed_time(ev_e1) / EMB_REPS
            t_emb_cold += ev_c0.elapsed_time(ev_c1) / EMB_TABLES
            if i8 is not None:
                t_i8 += ev_i0.elapsed_time(ev_i1) / GEMM_REPS
            for k, members in groups.items():
                for i in members:
                    t_quant[i] += gev[k][0].elapsed_time(gev[k][1]) / (len(members) * QUANT_REPS)
            for i in range(nl):
                t_gemm[i] += evs[i][1].elapsed_time(evs[i][2]) / GEMM_REPS
        # ---- the same step with its five independent jobs spread over five streams (reported beside `value`)
        overlapped_ms = None
        if not args.profile_mode and n_streams == 1:
            for _ in range(3):
                step(5)
            barrier()
            ev0.record(stream)
            for _ in range(args.steps):
                step(5)
            ev1.record(stream)
            barrier()
            overlapped_ms = ev0.elapsed_time(ev1) / args.steps
            step(1)  # leaves launches_per_step as counted for the timed configuration
            barrier()
    clocks = sampler.summary()
    if args.profile_mode:
        if rank == 0:
            print(json.dumps({"profile_mode": True, "ms_per_step": ms / args.steps, "steps": args.steps}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return 0

    ms = dist_util.max_over_ranks(ms, dev)
    ms_per_step = ms / args.steps
    value = dist_util.whole_job_rate(ops, world, ms_per_step) / 1e12

    # ---- end to end: host buffers, H2D of every input and D2H of every output inside the timed region
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    host_in = [torch.from_numpy(L["X"]).pin_memory() for L in layers]
    host_ids = ids.cpu().pin_memory()
    host_out = [torch.empty((L["M"], L["N"]), dtype=torch.float32).pin_memory() for L in layers]
    host_emb = torch.empty((M, H), dtype=torch.float32).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host_in) + host_ids.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in host_out) + host_emb.numel() * 4

    # Host-to-device copies, kernels and device-to-host copies run on three streams chained by events, so the two
    # copy directions and the compute overlap across the jobs of a step (and across steps).  A job's input buffer is
    # refilled only after the previous step's kernels have read it, its output only after the read-back has left.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    njobs = len(layers) + 1
    ev_in = [torch.cuda.Event() for _ in range(njobs)]
    ev_done = [torch.cuda.Event() for _ in range(njobs)]
    ev_out = [torch.cuda.Event() for _ in range(njobs)]
    for e_ in ev_done + ev_out:
        e_.record(stream)

    def e2e_step():
        jobs = [(ids, host_ids, emb_out, host_emb, lambda: q8.q8_embedding(ids, Eq, S_e, out=emb_out))]
        for L, hi, ho in zip(layers, host_in, host_out):
            jobs.append((L["Xd"], hi, L["Y"], ho,
                         lambda L=L: q8.q8_linear(L["Xd"], L["Wq"], L["S_w"], L["S_x"], L["bd"], L["act"], Y=L["Y"],
                                                  workspace=L["ws"])))
        for j, (d_in, h_in, d_out, h_out, run) in enumerate(jobs):
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_done[j])  # last step's kernel has consumed this input buffer
                d_in.copy_(h_in, non_blocking=True)
                ev_in[j].record(s_in)
            stream.wait_event(ev_in[j])
            stream.wait_event(ev_out[j])     # last step's read-back of this output buffer has finished
            run()
            ev_done[j].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[j])
                h_out.copy_(d_out, non_blocking=True)
                ev_out[j].record(s_out)

    def e2e_join():
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)

    e2e_step()
    e2e_join()
    barrier()
    ev0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e2e_join()
    ev1.record(stream)
    barrier()
    e2e_ms = ev0.elapsed_time(ev1)
    e2e_ms = dist_util.max_over_ranks(e2e_ms, dev)
    e2e_value = dist_util.whole_job_rate(ops, world, e2e_ms / e2e_steps) / 1e12

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel (the tcgen05 GEMM, launched once per FC layer)
    peaks, peak_kind = load_peaks()
    # Burst peak when the SM clock stayed at its maximum during the timed region (short step, no power cap),
    # the sustained one when the clock sagged under the power cap.
    at_max_clock = bool(clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    peak_key = "bf16_tflops" if at_max_clock else "bf16_tflops_sustained"
    sm_hz = float(clocks.get("sm_mhz") or 1965.0) * 1e6  # SM clock sampled while the timed region ran
    int8_peak = float(peaks.get(peak_key, FALLBACK_PEAKS[peak_key])) * NOMINAL_INT8_OVER_BF16
    int8_peak_sustained = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])) * NOMINAL_INT8_OVER_BF16
    hbm_peak = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    gemm_ms = [t / ksteps for t in t_gemm]
    quant_ms = [t / ksteps for t in t_quant]
    gemm_ops = [2.0 * L["M"] * L["N"] * L["K"] for L in layers]
    gemm_bytes = [L["M"] * L["K"] + L["N"] * L["K"] + 4 * L["N"] + 4 * L["M"] * L["N"] for L in layers]
    achieved = sum(gemm_ops) / (sum(gemm_ms) * 1e-3) / 1e12
    by_layer = []
    for L, gm, qm, go, gb in zip(layers, gemm_ms, quant_ms, gemm_ops, gemm_bytes):
        by_layer.append({
            "layer": L["name"], "M": L["M"], "K": L["K"], "N": L["N"],
            "gemm_us": gm * 1e3, "gemm_tops": go / (gm * 1e-3) / 1e12, "gemm_frac_int8_peak": go / (gm * 1e-3) / 1e12 / int8_peak,
            "gemm_gbs": gb / (gm * 1e-3) / 1e9, "gemm_frac_hbm": gb / (gm * 1e-3) / 1e9 / hbm_peak,
            "quantize_us": qm * 1e3, "quantize_gbs": 5.0 * L["M"] * L["K"] / (qm * 1e-3) / 1e9,
            "quantize_frac_hbm": 5.0 * L["M"] * L["K"] / (qm * 1e-3) / 1e9 / hbm_peak,
        })
    # Bytes that cross between L2 and the SMs per launch with 256 x 256 pair tiles: every tile pulls its 256 rows
    # of X_q and of W_q over the whole K, and pushes its fp32 block out once.
    fabric_bytes = []
    for L in layers:
        tiles_m, tiles_n = -(-L["M"] // 256), -(-L["N"] // 256)
        fabric_bytes.append(tiles_m * tiles_n * 512 * L["K"] + 4 * L["M"] * L["N"])
    # Issue-bound Int8 rate of the tensor cores on this device (operands resident in shared memory), measured now
    mma_peak = None
    if world == 1:
        st_word = torch.zeros(1, dtype=torch.int32, device=dev)
        burst = q8.q8_measure_int8_mma_peak(2, 0.02, dev_status=st_word)
        sustained = q8.q8_measure_int8_mma_peak(2, 0.5, dev_status=st_word)
        mma_peak = {
            "burst_tops": burst["tops"], "burst_ms": burst["elapsed_ms"], "sustained_tops": sustained["tops"],
            "sustained_ms": sustained["elapsed_ms"], "status": int(st_word.item()),
            "frac_of_burst": achieved / burst["tops"], "frac_of_sustained": achieved / sustained["tops"],
            "what": "tcgen05.mma cta_group::2 kind::i8 256x256x32 issued back to back on all SM pairs, operands resident "
                    "in shared memory, no loads or stores (q8_measure_int8_mma_peak)",
        }
    # One-directional HBM rates measured now (a copy moves a byte in per byte out; the fp32 output of an FC layer
    # is almost pure store traffic): the floor of a layer is the slower of its MMAs at the Int8 peak and its
    # 4 M N output bytes at the store-only rate.
    hbm_dir = None
    if world == 1:
        probe = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
        st_r = q8.q8_measure_hbm_peak(probe, store=True, repeats=10)
        ld_r = q8.q8_measure_hbm_peak(probe, store=False, repeats=10)
        del probe
        t_floor = []
        for L, go, bl in zip(layers, gemm_ops, by_layer):
            y_bytes = 4.0 * L["M"] * L["N"]
            t_tensor = go / (int8_peak * 1e12)
            t_store = y_bytes / (st_r["gbs"] * 1e9)
            t_floor.append(max(t_tensor, t_store))
            bl["gemm_y_store_gbs"] = y_bytes / (bl["gemm_us"] * 1e-6) / 1e9
            bl["gemm_frac_hbm_store"] = bl["gemm_y_store_gbs"] / st_r["gbs"]
            bl["gemm_floor_us"] = t_floor[-1] * 1e6
            bl["gemm_floor_bound"] = "hbm_store" if t_store > t_tensor else "tensor"
            bl["gemm_frac_of_floor"] = t_floor[-1] * 1e6 / bl["gemm_us"]
        hbm_dir = {
            "store_gbs": st_r["gbs"], "load_gbs": ld_r["gbs"], "copy_gbs": hbm_peak,
            "gemm_floor_us": sum(t_floor) * 1e6, "gemm_us": sum(gemm_ms) * 1e3,
            "gemm_frac_of_floor": sum(t_floor) / (sum(gemm_ms) * 1e-3),
            "what": "store-only and load-only rates of a grid-stride 16-byte kernel over 1 GiB (q8_measure_hbm_peak); per "
                    "layer floor = max(2MNK / Int8 peak, 4MN / store-only rate)",
        }
    # What L2 can feed the SMs through TMA, measured now on an L2-resident matrix of the first layer's operand shape
    l2_probe = None
    n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    if world == 1:
        pm = torch.zeros((4096, 1024), dtype=torch.int8, device=dev)
        r4 = q8.q8_measure_l2_operand_peak(pm, 4096, 1024, boxes_per_sm=2048, producers=4)
        r1 = q8.q8_measure_l2_operand_peak(pm, 4096, 1024, boxes_per_sm=2048, producers=1)
        del pm
        l2_probe = {"tbs_all_sms_4_issuing_warps": r4["gbs"] / 1e3, "gbs_per_sm_4_issuing_warps": r4["gbs"] / n_sms,
                    "gbs_per_sm_1_issuing_warp": r1["gbs"] / n_sms,
                    "needed_gbs_per_sm_at_full_int8_rate": 64.0 * sm_hz / 1e9,
                    "what": "q8_measure_l2_operand_peak: 128-row x 128-byte boxes, 12 stages in flight per SM"}
    emb_ms = t_emb / ksteps
    emb_cold_ms = t_emb_cold / ksteps
    emb_bytes = 5.0 * M * H + 4.0 * M
    if i8 is not None:
        L = layers[i8]
        im = t_i8 / ksteps
        go = 2.0 * L["M"] * L["N"] * L["K"]
        gb = L["M"] * L["K"] + L["N"] * L["K"] + 4 * L["N"] + L["M"] * L["N"]
        t_tensor = go / (int8_peak * 1e12)
        by_layer.append({
            "layer": "ffn1_int8_out", "M": L["M"], "K": L["K"], "N": L["N"], "gemm_us": im * 1e3,
            "gemm_tops": go / (im * 1e-3) / 1e12, "gemm_frac_int8_peak": go / (im * 1e-3) / 1e12 / int8_peak,
            "gemm_gbs": gb / (im * 1e-3) / 1e9, "gemm_frac_hbm": gb / (im * 1e-3) / 1e9 / hbm_peak,
            "gemm_floor_us": t_tensor * 1e6, "gemm_floor_bound": "tensor", "gemm_frac_of_floor": t_tensor / (im * 1e-3),
            "note": "q8_linear_q_requant: FFN1 with GELU emitting only Int8 at FFN2's scale (1 byte per output); not part of the step",
        })
    roofline = {
        "kernel": "gemm_tcgen05_kernel (4 launches per step, one per FC layer)",
        "bound": "tensor", "achieved": achieved, "peak": int8_peak, "unit": "TOP/s", "frac": achieved / int8_peak,
        "traffic": (sum(GEMM_DRAM_TRAFFIC[args.workload][L["name"]] for L in layers) / len(layers)
                    if args.workload in GEMM_DRAM_TRAFFIC else None),
        "traffic_note": "mean DRAM bytes per GEMM launch from ncu (profiles/gemm_tcgen05_dram_traffic_m24576.md); "
                        "algorithmic mean is %.0f" % (sum(gemm_bytes) / len(gemm_bytes)),
        "peak_source": f"2 x {peak_key} of {peak_kind} (nominal int8:bf16 dense ratio); "
                       + ("burst figure: SM clock at max in the timed region" if at_max_clock else "sustained figure: SM clock below max"),
        "frac_of_sustained_peak": achieved / int8_peak_sustained,
        "frac_of_nominal_4500": achieved / 4500.0,
        "int8_mma_issue_peak": mma_peak,
        "hbm_one_directional": hbm_dir,
        "l2_sm_traffic": {
            "bytes_per_launch_mean": sum(fabric_bytes) / len(fabric_bytes),
            "achieved_tbs": sum(fabric_bytes) / (sum(gemm_ms) * 1e-3) / 1e12,
            "by_layer_tbs": {L["name"]: fb / (gm * 1e-3) / 1e12 for L, fb, gm in zip(layers, fabric_bytes, gemm_ms)},
            "l2_operand_probe": l2_probe,
            "note": "operand re-loads of the 256 x 256 pair tiles plus the fp32 output, all through L2.  L2 itself is not the "
                    "limit: the probe (TMA loads of the GEMM's operand boxes by every SM, nothing else running, measured "
                    "now) delivers well above the 64 B/clk/SM the main loop asks for at the full Int8 rate",
        },
        "sm_side_limits": {
            "write_port_bytes_per_clk_per_sm": 32,
            "y_store_us_at_write_port": {L["name"]: 4.0 * L["M"] * L["N"] / (n_sms * 32.0 * sm_hz) * 1e6 for L in layers},
            "main_loop_only_us": {"qkv": 44.6, "attn_out": 18.7, "ffn1": 58.3, "ffn2": 66.4} if args.workload == "bert_large_fc" else None,
            "note": "an SM writes to L2 at no more than 32 bytes per clock (ncu: l1tex__m_l1tex2xbar_write_bytes peak), "
                    "whether by TMA store or by st.global, so the fp32 output of a layer occupies that port for "
                    "y_store_us_at_write_port (at the SM clock sampled in this run); measured kernel times are close to "
                    "main_loop_only_us (the same kernel with the epilogue reduced to handing the accumulator back, an "
                    "experimental build, graph-replayed) plus that port time, i.e. the two do not overlap.  The main loop alone runs at "
                    "about three quarters of the issue-bound Int8 rate: TMA writes 64 B/clk/SM into shared memory while "
                    "the tensor cores read 64 B/clk/SM from it (with no loads the same loop takes 54.5 us on FFN2, with "
                    "only the B tiles 56.3, with both operands 66.4)",
        },
        "note": "GEMM times: CUDA events around a graph replay of %d back-to-back launches of the layer (X_q just written by the quantise "
                "pass, output streamed to HBM); quantise times: events around the back-to-back group of equal-sized layers "
                "(a single launch for FFN2's input); embedding: events around %d launches that alternate between two output buffers; "
                "all replayed from CUDA graphs unless --no-graph" % (GEMM_REPS, EMB_REPS),
        "by_layer": by_layer,
        "embedding": {"us": emb_ms * 1e3, "gbs": emb_bytes / (emb_ms * 1e-3) / 1e9,
                      "frac_hbm": emb_bytes / (emb_ms * 1e-3) / 1e9 / hbm_peak,
                      "l2_cold": {"us": emb_cold_ms * 1e3, "gbs": emb_bytes / (emb_cold_ms * 1e-3) / 1e9,
                                  "frac_hbm": emb_bytes / (emb_cold_ms * 1e-3) / 1e9 / hbm_peak,
                                  "note": "%d gathers in a row, each from its own copy of the table (together larger than L2), "
                                          "alternating between two output buffers" % EMB_TABLES}},
    }

    # ---- CPU oracle on a bounded sample of the same workload (rank 0, N=1 only)
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import q8_oracle as o
        rows = min(args.cpu_rows, M)
        t0 = time.perf_counter()
        for L in layers:
            Wq_h = L["Wq"].cpu().numpy()
            o.linear(L["X"][:rows], Wq_h, float(L["S_w"].item()), float(L["S_x"].item()), L["b"], L["act"])
        dt = time.perf_counter() - t0
        sample_ops = sum(2.0 * rows * L["N"] * L["K"] for L in layers)
        cpu_baseline = {
            "value": sample_ops / dt / 1e12, "unit": "TOPS", "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"first {rows} of {M} token rows of each of the 4 FC layers, once ({dt:.1f} s)",
        }

    graph_replayed = step_graph is not None
    # ---- whole encoder forwards (tokens/s): int8 embeddings, every FC quantised, attention / LayerNorm in fp32
    encoder = small = None
    if world == 1 and not args.no_encoder:
        for L in layers:
            L.clear()
        del host_in, host_out, host_emb, emb_out, emb_out2, gemm_graphs, quant_graphs, emb_graph, step_graph
        del Eq_copies, emb_cold_graph, i8_graph, Yq_i8
        torch.cuda.empty_cache()
        encoder = measure_encoders(args, torch, q8)
        small = measure_small_cases(args, torch, q8)

    srt = sorted(per_step_ms)
    line = {
        "metric": "q8_linear_int8_tops", "value": value, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        # per-kernel microseconds first, so that a truncated copy of this line still shows every layer
        "kernel_us": dict([(b["layer"], round(b["gemm_us"], 2)) for b in by_layer]
                          + [("quantize_" + b["layer"], round(b["quantize_us"], 2)) for b in by_layer if "quantize_us" in b]
                          + [("embedding", round(emb_ms * 1e3, 2)), ("embedding_l2_cold", round(emb_cold_ms * 1e3, 2))]),
        "gemm_frac_nominal_int8_4500": dict((b["layer"], round(b["gemm_tops"] / 4500.0, 4)) for b in by_layer),
        "step_us": {"mean_of_timed_region": ms_per_step * 1e3,
                    "median": (statistics.median(srt) * 1e3 if srt else None), "best": (srt[0] * 1e3 if srt else None),
                    "samples": len(srt), "tops_at_median": (ops * world / (statistics.median(srt) * 1e-3) / 1e12 if srt else None)},
        "config": {
            "workload": args.workload, "description": desc, "tokens_per_step": M * world,
            "tokens_per_s": M * world / (ms_per_step * 1e-3),
            "l2": "inputs larger than L2 (each step reads ~0.9 GB and writes ~1.0 GB; L2 is 126 MB)",
            "step": "q8_embedding + 4 x q8_linear (quantise, tcgen05 GEMM, fused epilogue), static scales",
            "streams": n_streams,
            "launch": ("one CUDA graph replay per step" if graph_replayed else "eager launches"),
            "eager_ms_per_step": eager_ms,
            "overlapped": (None if overlapped_ms is None else {
                "streams": 5, "ms_per_step": overlapped_ms, "value": ops / (overlapped_ms * 1e-3) / 1e12, "unit": "TOPS",
                "note": "same step, its five independent jobs on five streams (HBM-bound passes overlap the GEMMs)"}),
        },
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TOPS", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                "note": "pinned host buffers; H2D copies, kernels and D2H copies on three streams chained by events"},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline,
        "cpu_baseline": cpu_baseline,
        "encoder": encoder,
        "small_cases": small,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def profile_encoder_kernel(args, torch, q8):
    """--profile-mode --encoder-kernel K: a few launches of one FP32 support kernel of the encoder (attention or
    residual + LayerNorm) on seeded synthetic data, for an ncu capture of that kernel alone."""
    B, S, heads, H = args.profile_batch, args.profile_seq, args.profile_heads, args.profile_heads * 64
    g = torch.Generator(device="cuda").manual_seed(1)
    if args.encoder_kernel == "attention":
        qkv = torch.randn((B * S, 3 * H), device="cuda", generator=g)
        ctx = torch.empty((B * S, H), device="cuda")
        fn = lambda: q8.q8_attention(qkv, B, S, heads, ctx=ctx)
        work, unit = 4.0 * B * heads * S * S * 64, "TFLOP/s"
    else:
        x = torch.randn((B * S, H), device="cuda", generator=g)
        r = torch.randn((B * S, H), device="cuda", generator=g)
        out = torch.empty_like(x)
        fn = lambda: q8.q8_add_layernorm(x, r, out=out)
        work, unit = 12.0 * B * S * H, "TB/s"
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(max(args.steps, 1)):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / max(args.steps, 1)
    print(json.dumps({"profile_mode": True, "encoder_kernel": args.encoder_kernel, "batch": B, "seq": S, "heads": heads,
                      "us_per_call": ms * 1e3, "rate": work / (ms * 1e-3) / 1e12, "unit": unit}), flush=True)
    return 0


def measure_small_cases(args, torch, q8):
    """The two smaller workload configurations, timed as back-to-back calls (their data fits in L2, so these are
    L2-warm, launch-latency-dominated figures; reported in microseconds rather than against a roofline)."""
    out = {}
    dev = torch.device("cuda", torch.cuda.current_device())

    def timed(fn, reps):
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e3

    # config 1: one layer, X [128 x 768], dynamic scale (Sec. 4.1): absmax, scale, quantise, GEMM
    X = torch.from_numpy(synth.activation(128, 768, synth.seed_for(1, 0))).to(dev)
    Wq, S_w = q8.q8_quantize_weight(torch.from_numpy(synth.weight(768, 768, synth.seed_for(1, 1))).to(dev))
    b = torch.from_numpy(synth.bias(768, synth.seed_for(1, 2))).to(dev)
    Y = torch.empty((128, 768), device=dev)
    ws = q8.new_workspace(128, 768, 768, dev)
    us = timed(lambda: q8.q8_linear(X, Wq, S_w, None, b, 0, Y=Y, workspace=ws), 200)
    info = q8.q8_last_launch_info()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        q8.q8_linear(X, Wq, S_w, None, b, 0, Y=Y, workspace=ws)
    us_graph = timed(graph.replay, 200)
    out["single_layer_128x768x768_dynamic"] = {"us_per_call": us, "us_per_call_cuda_graph": us_graph,
                                               "launches": info["launches"], "block_n": info["block_n"],
                                               "grid": info["grid"], "tops": 2.0 * 128 * 768 * 768 / us_graph / 1e6}
    del graph
    # config 2: BERT-Base FC set, M = 4096, static scales
    M, layers = make_layers(2, synth.BERT_BASE)
    for L in layers:
        L["Xd"] = torch.from_numpy(L["X"]).to(dev)
        L["bd"] = torch.from_numpy(L["b"]).to(dev)
        L["Wq"], L["S_w"] = q8.q8_quantize_weight(torch.from_numpy(L["W"]).to(dev))
        st = q8.new_calibrate_state(dev)
        q8.q8_calibrate(torch.from_numpy(L["calib"]).to(dev), 0.9999, st)
        L["S_x"] = q8.calibrate_S_x(st).clone()
        L["Y"] = torch.empty((M, L["N"]), device=dev)
        L["ws"] = q8.new_workspace(M, L["N"], L["K"], dev)

    def step():
        for L in layers:
            q8.q8_linear(L["Xd"], L["Wq"], L["S_w"], L["S_x"], L["bd"], L["act"], Y=L["Y"], workspace=L["ws"])
    us = timed(step, 100)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    us_graph = timed(graph.replay, 100)
    out["bert_base_fc_set_m4096"] = {"us_per_step": us, "us_per_step_cuda_graph": us_graph,
                                     "tops": total_ops(layers) / us_graph / 1e6,
                                     "note": "the same buffers every step; a step touches ~230 MB (88 MB of fp32 inputs, 22 MB of "
                                             "X_q, 113 MB of fp32 outputs, 7 MB of weights), more than the 126 MB of L2, so "
                                             "only the weights are warm"}
    return out


def measure_encoders(args, torch, q8):
    """Tokens/s of whole BERT-Base (32 x 128) and BERT-Large (64 x 384) encoder forwards with static scales,
    plus where the time goes (CUDA events around every call of one extra forward)."""
    from paper_1910_06188_b200 import encoder as enc_mod

    out = {}
    for name, dims, cfg in (("bert_base_32x128", synth.BERT_BASE, 3), ("bert_large_64x384", synth.BERT_LARGE, 5)):
        B, S = dims["batch"], dims["seq"]
        T = B * S
        enc = enc_mod.Q8BertEncoder(dims, config=cfg)
        ids = enc_mod.random_ids(T, dims["vocab"], cfg)
        enc.forward(ids, B, S, scales="calibrate")
        for _ in range(3):
            enc.forward(ids, B, S)
        torch.cuda.synchronize()
        reps = args.encoder_steps
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            enc.forward(ids, B, S)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        # the same forward with every quantiser fused into its producer (bit-identical result)
        for _ in range(2):
            enc.forward_fused(ids, B, S)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            enc.forward_fused(ids, B, S)
        e1.record()
        torch.cuda.synchronize()
        ms_fused = e0.elapsed_time(e1) / reps
        # ... and replayed from a CUDA graph (removes the host launch cost, which dominates the small model)
        graph, _ = enc.capture(ids, B, S)
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        ms_graph = e0.elapsed_time(e1) / reps
        del graph
        # dynamic quantisation (Sec. 4.1): every FC computing its own max|x|, against producers folding it
        dyn = {}
        for label, run in (("dynamic", lambda: enc.forward(ids, B, S, scales="dynamic")),
                           ("dynamic_fused_absmax", lambda: enc.forward_dynamic_fused(ids, B, S))):
            for _ in range(2):
                run()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(reps):
                run()
            e1.record()
            torch.cuda.synchronize()
            dyn[label] = e0.elapsed_time(e1) / reps
        codes = enc.poll()
        # breakdown: time the three kinds of calls of one forward
        shares = {"q8_linear": 0.0, "attention_fp32": 0.0, "layernorm_embedding": 0.0}
        orig = {k: getattr(q8, k) for k in ("q8_linear", "q8_attention", "q8_add_layernorm", "q8_embedding")}
        evs = []

        def timed(fn, key):
            def wrapper(*a, **k):
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a0.record()
                r = fn(*a, **k)
                a1.record()
                evs.append((key, a0, a1))
                return r
            return wrapper
        try:
            q8.q8_linear = timed(orig["q8_linear"], "q8_linear")
            q8.q8_attention = timed(orig["q8_attention"], "attention_fp32")
            q8.q8_add_layernorm = timed(orig["q8_add_layernorm"], "layernorm_embedding")
            q8.q8_embedding = timed(orig["q8_embedding"], "layernorm_embedding")
            enc.forward(ids, B, S)
            torch.cuda.synchronize()
        finally:
            for k, fn in orig.items():
                setattr(q8, k, fn)
        for key, a0, a1 in evs:
            shares[key] += a0.elapsed_time(a1)
        fc_ops = enc.L * sum(2.0 * T * N * K for _, K, N, _ in synth.fc_set(enc.H, enc.F))
        # CPU oracle beside it (part of the cpu_baseline leg): one encoder layer of this model on one sequence
        # (batch 1), timed on the host cores and extrapolated linearly to the whole model.
        cpu_oracle = None
        if not args.no_cpu_baseline:
            from oracle import q8_oracle as o
            f32 = lambda a: np.asarray(a, dtype=np.float32)
            lw = {n: (enc.layers[0][n]["Wq"].cpu().numpy(), float(enc.layers[0][n]["S_w"].item()),
                      float(q8.calibrate_S_x(enc.layers[0][n]["state"]).item()), enc.layers[0][n]["b"].cpu().numpy())
                  for n in ("qkv", "attn_out", "ffn1", "ffn2")}
            h = synth.activation(S, enc.H, synth.seed_for(cfg, 95))
            lin = lambda n, X, act: f32(o.linear(X, lw[n][0], lw[n][1], lw[n][2], lw[n][3], act)["y"])
            t0 = time.perf_counter()
            qkv = lin("qkv", h, 0)
            ctx = f32(o.attention(qkv, 1, S, enc.heads))
            h1 = f32(o.add_layernorm(lin("attn_out", ctx, 0), h, eps=enc_mod.LN_EPS))
            f2 = lin("ffn2", lin("ffn1", h1, 1), 0)
            o.add_layernorm(f2, h1, eps=enc_mod.LN_EPS)
            dt = time.perf_counter() - t0
            cpu_oracle = {"one_layer_one_sequence_s": dt, "tokens_per_s_extrapolated": S / (dt * enc.L),
                          "cores": os.cpu_count(), "kind": "oracle",
                          "sample": f"layer 0 on one sequence of {S} tokens; extrapolated linearly to {enc.L} layers"}
        out[name] = {
            "tokens_per_s": T / (ms * 1e-3), "ms_per_forward": ms, "layers": enc.L, "tokens": T,
            "tokens_per_s_fused_requant": T / (ms_fused * 1e-3), "ms_per_forward_fused_requant": ms_fused,
            "tokens_per_s_fused_cuda_graph": T / (ms_graph * 1e-3), "ms_per_forward_fused_cuda_graph": ms_graph,
            "ms_per_forward_dynamic": dyn["dynamic"], "ms_per_forward_dynamic_fused_absmax": dyn["dynamic_fused_absmax"],
            "tokens_per_s_dynamic_fused_absmax": T / (dyn["dynamic_fused_absmax"] * 1e-3),
            "gpu_launches_per_forward": enc.launches_per_forward(),
            "gpu_launches_per_forward_fused_requant": enc.launches_per_forward(fused=True),
            "status": [list(c) for c in codes],
            "ms_by_kind": shares, "q8_linear_tops_inside_forward": fc_ops / (shares["q8_linear"] * 1e-3) / 1e12,
            "int8_parameter_bytes": enc.memory_bytes_int8(),
            "cpu_oracle": cpu_oracle,
        }
        del enc
        torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="bert_large_fc")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-rows", type=int, default=24576,
                    help="token rows per layer for the cpu_baseline sample (default: the whole workload once, ~10 s)")
    ap.add_argument("--reference-rows", type=int, default=0,
                    help="token rows per layer per step for --impl reference (0 = the whole workload, as the GPU arm)")
    ap.add_argument("--reference-budget-s", type=float, default=150.0,
                    help="--impl reference cuts its step count so that the run stays within this many seconds")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-encoder", action="store_true", help="skip the whole-encoder tokens/s measurement")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of CUDA graph replays")
    ap.add_argument("--encoder-steps", type=int, default=5)
    ap.add_argument("--streams", type=int, default=1,
                    help="streams used inside a step for the independent layers of the FC set (1 = serial)")
    ap.add_argument("--layers", default="", help="comma list of FC layers to keep (qkv,attn_out,ffn1,ffn2); default all")
    ap.add_argument("--profile-mode", action="store_true",
                    help="only warm-up + timed steps (no per-kernel pass, e2e or CPU baseline): for ncu captures")
    ap.add_argument("--encoder-kernel", choices=["attention", "layernorm"], default="",
                    help="with --profile-mode: launch only this FP32 support kernel of the encoder (--steps times)")
    ap.add_argument("--profile-int8-out", action="store_true",
                    help="with --profile-mode: the FC layers emit only Int8 (q8_linear_requant), for captures of that epilogue")
    ap.add_argument("--profile-batch", type=int, default=8)
    ap.add_argument("--profile-seq", type=int, default=384)
    ap.add_argument("--profile-heads", type=int, default=16)
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
