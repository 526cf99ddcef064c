#!/usr/bin/env python
"""Benchmark of the quantized-pruning hot path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input: the
prefill-side compression (window scores -> top-k -> gather+quantize+pack) of every layer,
followed by every decode step's attention over the packed cache of every layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is the decode-attention throughput in GB/s of
algorithmic packed-cache bytes (codes + scale/zero) with everything resident in HBM; `e2e`
is the same quantity with the step's inputs coming from pinned host memory and the results
going back, through the same C-ABI calls.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2412_12706_b200 import shard, synth

METRIC = "decode_attn_hbm_gbs"
UNIT = "GB/s"
DEFAULT_WORKLOAD = synth.LLAMA8B_8K.name
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of the dominant (decode) kernel from an ncu capture, valid only for the exact
# kernel sources it was taken on: {"sha256": <hash of DECODE_KERNEL_SOURCES>, "workload": name,
# "bytes_per_launch": dram__bytes_read.sum + dram__bytes_write.sum}
NCU_TRAFFIC: dict = {
    "sha256": "fe3610834b63199d2b039d77863582141288ce877979e8ba2832af91138c1d4c",
    "workload": "llama3-8b-8k-b1-4bit",
    # captured on a 4-sequence call, the launch shape of the default run (336.81 MB read + 5.95 MB written per
    # launch, mean of two launches); other group sizes scale it: the traffic is proportional to the tiles streamed
    "bytes_per_launch_per_sequence": (336810112 + 5953024) / 4,
}

KERNELS_PER_COMPRESS = 6      # sweep 1, row-stat merge, sweep 2, pool, top-k, gather+quantize
KERNELS_PER_DECODE_CALL = 2   # split-K attention, merge
DECODE_KERNEL_SOURCES = ("qp_decode.cu", "qp_decode_mma.cu", "qp_decode_mma2.cu", "qp_mma.cuh")


def packed_bytes(wl: synth.Workload, layer: int) -> int:
    """Algorithmic bytes one decode step reads for one layer: codes plus fp16 scale and zero."""
    n, b, g = wl.n_keep(layer), wl.bits, wl.group
    elems = wl.batch * wl.n_kv_heads * n * wl.head_dim * 2            # K and V
    return elems * 2 if b == 16 else elems * (b + 32 // g) // 8


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(gpu_index)], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(names, r[5:9]):
                if val.strip().lower() == "active":
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- reference arm

def oracle_sample(wl: synth.Workload, steps: int, warmup: int):
    """The CPU oracle, as it stands, on a bounded sample of the workload (sized for roughly
    10-20 s of host time per step): the first few layers of one sequence, each compressed once
    and attended for `dec` decode steps."""
    from oracle import qp_oracle as orc
    u16 = synth.bits_u16
    dec = 8
    if wl.batch > 1:                                   # large configurations: one batch entry only
        wl = synth.dataclasses.replace(wl, batch=1)
    macs = wl.n_kv_heads * (wl.n_q_heads // wl.n_kv_heads) * wl.w * wl.L * wl.head_dim
    n_lay = max(1, min(wl.n_layers, 16, int(2e10 // macs)))
    layers = []
    for l in range(n_lay):
        k, v = synth.make_kv(wl, l)
        layers.append((u16(k), u16(v), u16(synth.make_q_win(wl, l)),
                       [u16(synth.make_q_dec(wl, l, s)) for s in range(dec)]))
    t_comp, t_dec = [], []
    for it in range(warmup + steps):
        tc = td = 0.0
        for l, (kb, vb, qwb, qs) in enumerate(layers):
            t0 = time.perf_counter()
            pk, kept, _ = orc.compress_layer(kb, vb, qwb, wl.layer_budget_bits(l), wl.bits, wl.group, wl.pool)
            t1 = time.perf_counter()
            for s in range(dec):
                kd, vd = orc.dequantize(pk, wl.head_dim)    # the paper's decode dequantizes, then attends
                orc.decode(qs[s], kd, vd)
            t2 = time.perf_counter()
            tc += t1 - t0; td += t2 - t1
        if it >= warmup:
            t_comp.append(tc); t_dec.append(td)
    bytes_dec = sum(packed_bytes(wl, l) for l in range(n_lay)) * dec
    return {
        "decode_gbs": bytes_dec / statistics.mean(t_dec) / 1e9,
        "compress_tokens_per_s": wl.batch * wl.L / (statistics.mean(t_comp) / n_lay * wl.n_layers),
        "ms_per_step": 1e3 * (statistics.mean(t_comp) + statistics.mean(t_dec)),
        "cores": orc.num_threads(),
        "sample": f"layers 0..{n_lay - 1} of one sequence (batch {wl.batch}): 1 compress_layer + {dec} decode "
                  f"steps per layer per step (of {wl.n_layers} layers x {wl.decode_steps} decode steps); "
                  f"compress tokens/s scaled to all {wl.n_layers} layers",
    }


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r = oracle_sample(wl, max(1, args.steps), max(0, min(args.warmup, 1)))
    line = {
        "impl": "reference", "metric": METRIC, "value": r["decode_gbs"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "sample": r["sample"]},
        "compress_tokens_per_s": r["compress_tokens_per_s"],
        "cpu_baseline": {"value": r["decode_gbs"], "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                         "sample": r["sample"]},
        "e2e": {"value": r["decode_gbs"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU arm

def run_gpu(args, wl):
    from paper_2412_12706_b200 import qp
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    qp.lib()
    qp.decode_overlap(not args.no_overlap)     # the decode steps are independent and nothing else runs between them

    n_seq, n_layers, n_dec = args.sequences, wl.n_layers, wl.decode_steps
    # sequences whose layers share one qp_decode_attn_layers call (independent problems, as in continuous batching)
    per_call = max(1, min(args.seqs_per_call, n_seq, qp.QP_MAX_LAYERS // n_layers))
    while n_seq % per_call:
        per_call -= 1
    Bt, Hq, Hkv, D, L, w = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.L, wl.w
    stream = torch.cuda.current_stream()

    # ---- inputs resident in HBM: every rank and every sequence has its own seed
    seqs = []
    for s in range(n_seq):
        wls = synth.dataclasses.replace(wl, seed=shard.sequence_seed(wl.seed, rank, n_seq, s))
        Ks, Vs, Qs = [], [], []
        for l in range(n_layers):
            k, v = synth.make_kv(wls, l, device=dev)
            Ks.append(k); Vs.append(v); Qs.append(synth.make_q_win(wls, l, device=dev))
        qdec = torch.stack([torch.stack([synth.make_q_dec(wls, l, t, device=dev) for l in range(n_layers)])
                            for t in range(n_dec)])              # [n_dec, n_layers, Bt, Hq, D]
        seqs.append({"K": Ks, "V": Vs, "Qw": Qs, "qdec": qdec})
    ws_c = torch.empty(qp.compress_workspace_bytes(Bt, Hq, Hkv, D, L, w), dtype=torch.uint8, device=dev)
    for sq in seqs:
        sq["cache"] = [qp.alloc_cache(Bt, Hq, Hkv, D, wl.bits, wl.group, wl.n_keep(l), dev) for l in range(n_layers)]
        sq["kept"] = [torch.empty((Bt, Hkv, wl.n_keep(l)), dtype=torch.int32, device=dev) for l in range(n_layers)]
        sq["out"] = torch.empty((n_layers, Bt, Hq, D), dtype=torch.bfloat16, device=dev)
        ws_d = qp.new_decode_workspace(sum(qp.decode_workspace_bytes(c) for c in sq["cache"]), dev)
        sq["ws_d"] = ws_d
        sq["batches"] = [qp.LayerBatch([sq["qdec"][t, l] for l in range(n_layers)], sq["cache"],
                                       [sq["out"][l] for l in range(n_layers)], ws_d) for t in range(min(n_dec, 8))]
    groups = []
    for g0 in range(0, n_seq, per_call):
        members = seqs[g0:g0 + per_call]
        ws_g = qp.new_decode_workspace(sum(m["ws_d"].numel() for m in members), dev)
        groups.append([qp.LayerBatch([m["qdec"][t, l] for m in members for l in range(n_layers)],
                                     [c for m in members for c in m["cache"]],
                                     [m["out"][l] for m in members for l in range(n_layers)], ws_g)
                       for t in range(n_dec)])

    dec_bytes_step = n_seq * n_dec * sum(packed_bytes(wl, l) for l in range(n_layers))
    dec_bytes_call = per_call * sum(packed_bytes(wl, l) for l in range(n_layers))
    ctx_tokens_step = n_seq * Bt * L

    def compress_all():
        for sq in seqs:
            for l in range(n_layers):
                qp.compress_layer(sq["K"][l], sq["V"][l], sq["Qw"][l], wl.layer_budget_bits(l), wl.bits, wl.group,
                                  wl.pool, sq["cache"][l], sq["kept"][l], ws_c)

    # the same work through qp_compress_layers: all layers of a sequence per call (one launch per stage)
    ws_cl = torch.empty(qp.compress_workspace_bytes(Bt * n_layers, Hq, Hkv, D, L, w), dtype=torch.uint8, device=dev) \
        if Bt * n_layers * Hkv <= 65535 and not args.no_compress_layers else None

    def compress_all_layers():
        budgets = [wl.layer_budget_bits(l) for l in range(n_layers)]
        for sq in seqs:
            qp.compress_layers(sq["K"], sq["V"], sq["Qw"], budgets, wl.bits, wl.group, wl.pool, sq["cache"], sq["kept"], ws_cl)

    def decode_all():
        # no event between the calls: consecutive decode calls overlap on the GPU (the next call's attention
        # kernel fills the SMs as this call's drains), and an event record in between would forbid that
        for t in range(n_dec):
            for grp in groups:       # consecutive launches touch different sequences' caches
                qp.decode_attn_layers(grp[t])
    n_calls_step = n_dec * len(groups)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        compress_all(); decode_all()
    barrier()

    sampler = ClockSampler(local) if rank == 0 else None
    ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = []
    barrier()
    t_begin = ev(); t_begin.record(stream)
    for _ in range(args.steps):
        a, b, c = ev(), ev(), ev()
        a.record(stream); compress_all(); b.record(stream); decode_all(); c.record(stream)
        marks.append((a, b, c))
    t_end = ev(); t_end.record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None

    total_ms = t_begin.elapsed_time(t_end)
    comp_ms = sum(a.elapsed_time(b) for a, b, c in marks)
    dec_ms = sum(b.elapsed_time(c) for a, b, c in marks)
    call_ms = dec_ms / (args.steps * n_calls_step)      # average launch duration over the timed decode phases

    # ---- compression with all layers of a sequence in one qp_compress_layers call
    comp_layers_ms = None
    if ws_cl is not None:
        compress_all_layers()
        k0, k1 = ev(), ev()
        k0.record(stream)
        for _ in range(3):
            compress_all_layers()
        k1.record(stream)
        torch.cuda.synchronize()
        comp_layers_ms = k0.elapsed_time(k1) / 3

    # ---- the same decode attention with one sequence per call (context for the batched figure)
    single_ms = None
    if per_call > 1:
        reps = 512
        for r in range(32):
            qp.decode_attn_layers(seqs[r % n_seq]["batches"][r % 8])
        s0, s1 = ev(), ev()
        s0.record(stream)
        for r in range(reps):
            qp.decode_attn_layers(seqs[r % n_seq]["batches"][r % 8])
        s1.record(stream)
        torch.cuda.synchronize()
        single_ms = s0.elapsed_time(s1) / reps

    # ---- and layer by layer: one qp_decode_attn call per layer, back to back, then the same chain replayed
    #      from a CUDA graph (what a model's decode loop would do between its other kernels)
    layer_ms = graph_ms = None
    if not args.no_layer_chain:
        sq0 = seqs[0]
        qs0, outs0 = sq0["qdec"][0], sq0["out"]
        ws_l = qp.new_decode_workspace(max(qp.decode_workspace_bytes(c) for c in sq0["cache"]), dev)

        def chain():
            for l in range(n_layers):
                qp.decode_attn(qs0[l], sq0["cache"][l], outs0[l], ws_l)
        for _ in range(3):
            chain()
        reps = 16
        c0, c1 = ev(), ev()
        c0.record(stream)
        for _ in range(reps):
            chain()
        c1.record(stream)
        torch.cuda.synchronize()
        layer_ms = c0.elapsed_time(c1) / reps
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            qp.decode_overlap(not args.no_overlap)
            chain()
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                chain()
            for _ in range(3):
                graph.replay()
            g0, g1 = ev(), ev()
            g0.record(side)
            for _ in range(reps):
                graph.replay()
            g1.record(side)
        torch.cuda.synchronize()
        graph_ms = g0.elapsed_time(g1) / reps

    # ---- generation loop: every decode step first appends the new token's key/value rows to every layer
    #      (qp_append_kv_layers; full tails are quantized into the caches) and then attends over packed
    #      tokens plus tail (qp_decode_attn_tail_layers).  Same grouping of sequences per call as above.
    gen = None
    if not args.no_generation:
        g_steps = 2 * wl.group + 8 if wl.bits < 16 else 72      # two flushes of every tail on the way
        room = 3 * wl.group if wl.bits < 16 else g_steps + 8
        gen_groups = []
        for g0 in range(0, n_seq, per_call):
            members = seqs[g0:g0 + per_call]
            caches, tails, kn, vn = [], [], [], []
            for i, m in enumerate(members):
                wls = synth.dataclasses.replace(wl, seed=shard.sequence_seed(wl.seed, rank, n_seq, g0 + i))
                for l in range(n_layers):
                    c, _ = qp.compress_layer(m["K"][l], m["V"][l], m["Qw"][l], wl.layer_budget_bits(l), wl.bits,
                                             wl.group, wl.pool, workspace=ws_c, n_cap=wl.n_keep(l) + room)
                    caches.append(c); tails.append(qp.alloc_tail(c))
                    a, b_ = synth.make_kv_new(wls, l, 0, device=dev)
                    kn.append(a); vn.append(b_)
            gen_groups.append(qp.GenBatch([m["qdec"][0, l] for m in members for l in range(n_layers)], kn, vn, caches,
                                          tails, [m["out"][l] for m in members for l in range(n_layers)]))
        gen_bytes0 = sum(gb.cache_arr[i].n_keep for gb in gen_groups for i in range(gb.n))

        def gen_step():
            for gb in gen_groups:
                qp.append_kv_layers(gb)
                qp.decode_attn_tail_layers(gb)
        for _ in range(4):
            gen_step()
        e0, e1 = ev(), ev()
        e0.record(stream)
        for _ in range(g_steps - 4):
            gen_step()
        e1.record(stream)
        torch.cuda.synchronize()
        gen_ms = e0.elapsed_time(e1) / ((g_steps - 4) * len(gen_groups))
        gen_bytes1 = sum(gb.cache_arr[i].n_keep for gb in gen_groups for i in range(gb.n))
        # packed bytes a call reads, averaged over the loop (the caches grow by a group at every flush)
        per_tok = Bt * Hkv * D * 2 * (2.0 if wl.bits == 16 else (wl.bits + 32 // wl.group) / 8)
        gen_call_bytes = 0.5 * (gen_bytes0 + gen_bytes1) * per_tok / len(gen_groups)
        gen = {"note": "per decode step and group of sequences: qp_append_kv_layers (new rows into the bf16 tails; "
                       "full tails quantized into the caches) + qp_decode_attn_tail_layers (packed tokens + tail)",
               "steps": g_steps - 4, "us_per_step_call": gen_ms * 1e3, "GB/s": gen_call_bytes / (gen_ms * 1e-3) / 1e9,
               "launches_per_step_call": "3 (4 on the steps that flush)"}
        del gen_groups

    # ---- end to end: host buffers in, host buffers out, through the same calls
    input_bytes = 2 * n_seq * n_layers * Bt * Hkv * L * D * 2
    # the host-buffer leg pins a copy of every input; keep it to workloads whose inputs are a few GB
    e2e = run_e2e(args, wl, qp, seqs, ws_c, dev, stream, dec_bytes_step, per_call) \
        if not args.no_e2e and input_bytes <= 10e9 else None

    def allmax(x: float) -> float:
        return shard.max_over_ranks(x, dist, dev)

    total_ms, comp_ms, dec_ms = allmax(total_ms), allmax(comp_ms), allmax(dec_ms)
    e2e_dec_ms = allmax(e2e["dec_ms"]) if e2e else None
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    steps = args.steps
    value = shard.whole_job_throughput(dec_bytes_step * steps, world, dec_ms * 1e-3) / 1e9
    peak, peak_kind = hbm_peak()
    achieved = dec_bytes_call / (call_ms * 1e-3) / 1e9
    sha = hashlib.sha256(b"".join(open(os.path.join(ROOT, "paper_2412_12706_b200", "csrc", f), "rb").read()
                                  for f in DECODE_KERNEL_SOURCES)).hexdigest()
    traffic = NCU_TRAFFIC["bytes_per_launch_per_sequence"] * per_call if NCU_TRAFFIC.get("sha256") == sha and \
        NCU_TRAFFIC.get("workload") == wl.name else None
    cpu = oracle_sample(wl, 1, 0) if world == 1 and not args.no_cpu_baseline else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": args.warmup,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "layers": n_layers, "batch": Bt, "q_heads": Hq, "kv_heads": Hkv,
                   "head_dim": D, "context": L, "window": w, "bits": wl.bits, "group": wl.group,
                   "n_keep": [wl.n_keep(0), wl.n_keep(n_layers - 1)], "decode_steps": n_dec,
                   "sequences_per_gpu": n_seq, "parallelism": f"replicas x{world}, no collective",
                   "decode_api": f"qp_decode_attn_layers: one launch pair per decode step over all layers of "
                                 f"{per_call} independent sequence(s) ({dec_bytes_call / 1e6:.0f} MB per call)",
                   "sequences_per_call": per_call,
                   "l2": f"decode rotates over {n_seq // per_call} group(s) of sequences "
                         f"({n_seq * dec_bytes_call / per_call / 1e6:.0f} MB of packed cache in all) so consecutive "
                         f"launches read different data; compress inputs {input_bytes / 1e9:.2f} GB"},
        "compress_tokens_per_s": world * ctx_tokens_step * steps / (comp_ms * 1e-3),
        "compress_ms_per_layer": comp_ms / (steps * n_seq * n_layers),
        "compress_layers_call": None if comp_layers_ms is None else {
            "note": f"qp_compress_layers: the {n_layers} layers of a sequence per call, one launch per stage",
            "ms_per_layer": comp_layers_ms / (n_seq * n_layers),
            "tokens_per_s": world * ctx_tokens_step / (comp_layers_ms * 1e-3)},
        "decode_us_per_call": call_ms * 1e3,
        "decode_single_sequence_call": None if single_ms is None else {
            "us_per_call": single_ms * 1e3, "GB/s": dec_bytes_call / per_call / (single_ms * 1e-3) / 1e9},
        "decode_layer_by_layer": None if layer_ms is None else {
            "note": "one sequence, one qp_decode_attn call per layer (its packed cache fits in L2 for small workloads)",
            "us_per_layer_call": layer_ms * 1e3 / n_layers,
            "GB/s": dec_bytes_call / per_call / (layer_ms * 1e-3) / 1e9,
            "cuda_graph_us_per_layer_call": graph_ms * 1e3 / n_layers,
            "cuda_graph_GB/s": dec_bytes_call / per_call / (graph_ms * 1e-3) / 1e9},
        "decode_with_append": gen,
        "decode_phase_ms_per_step": dec_ms / steps,
        "pct_of_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "kernel": "decode attention (split-K attention kernel + merge kernel, per call)",
                     "achieved": achieved,
                     "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic},
        "e2e": None if e2e is None else {
            "value": world * dec_bytes_step * e2e["steps"] / (e2e_dec_ms * 1e-3) / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
            "ms_per_step": e2e["total_ms"] / e2e["steps"],
            "compress_tokens_per_s": world * ctx_tokens_step * e2e["steps"] / (e2e["comp_ms"] * 1e-3)},
        "gpu_launches": steps * (n_seq * n_layers * KERNELS_PER_COMPRESS
                                 + (n_seq // per_call) * n_dec * KERNELS_PER_DECODE_CALL),
        "clocks": clocks,
    }
    if cpu is not None:
        line["cpu_baseline"] = {"value": cpu["decode_gbs"], "unit": UNIT, "cores": cpu["cores"], "kind": "oracle",
                                "sample": cpu["sample"], "compress_tokens_per_s": cpu["compress_tokens_per_s"]}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_e2e(args, wl, qp, seqs, ws_c, dev, stream, dec_bytes_step, per_call=1):
    """Same step, but every input starts in pinned host memory and every decode output is read
    back: K, V, Q_win are uploaded layer by layer before qp_compress_layer, each decode step
    uploads its queries and downloads its outputs."""
    n_layers, n_dec = wl.n_layers, wl.decode_steps
    hK = [[k.cpu().pin_memory() for k in sq["K"]] for sq in seqs]
    hV = [[v.cpu().pin_memory() for v in sq["V"]] for sq in seqs]
    hQ = [[q.cpu().pin_memory() for q in sq["Qw"]] for sq in seqs]
    dK, dV, dQ = torch.empty_like(seqs[0]["K"][0]), torch.empty_like(seqs[0]["V"][0]), torch.empty_like(seqs[0]["Qw"][0])
    # decode: the queries and the outputs of the sequences of one call are one contiguous block on either side,
    # so a call costs one upload and one download
    groups = []
    for g0 in range(0, len(seqs), per_call):
        ids = list(range(g0, g0 + per_call))
        hq_g = torch.stack([seqs[i]["qdec"] for i in ids], dim=1).cpu().pin_memory()     # [n_dec, per_call, layers, Bt, Hq, D]
        dq_g = torch.empty_like(hq_g[0], device=dev)
        dout_g = torch.empty_like(dq_g)
        hout_g = torch.empty_like(hq_g).pin_memory()
        ws_g = torch.empty(sum(seqs[i]["ws_d"].numel() for i in ids), dtype=torch.uint8, device=dev)
        batch = qp.LayerBatch([dq_g[j, l] for j in range(per_call) for l in range(n_layers)],
                              [c for i in ids for c in seqs[i]["cache"]],
                              [dout_g[j, l] for j in range(per_call) for l in range(n_layers)], ws_g)
        groups.append((hq_g, dq_g, dout_g, hout_g, batch))
    h2d = sum(t.numel() * 2 for per in (hK, hV, hQ) for s in per for t in s) + sum(g[0].numel() * 2 for g in groups)
    d2h = sum(g[3].numel() * 2 for g in groups)

    def step():
        a = torch.cuda.Event(enable_timing=True); a.record(stream)
        for i, sq in enumerate(seqs):
            for l in range(n_layers):
                dK.copy_(hK[i][l], non_blocking=True); dV.copy_(hV[i][l], non_blocking=True)
                dQ.copy_(hQ[i][l], non_blocking=True)
                qp.compress_layer(dK, dV, dQ, wl.layer_budget_bits(l), wl.bits, wl.group, wl.pool,
                                  sq["cache"][l], sq["kept"][l], ws_c)
        b = torch.cuda.Event(enable_timing=True); b.record(stream)
        for t in range(n_dec):
            for hq_g, dq_g, dout_g, hout_g, batch in groups:
                dq_g.copy_(hq_g[t], non_blocking=True)
                qp.decode_attn_layers(batch)
                hout_g[t].copy_(dout_g, non_blocking=True)
        c = torch.cuda.Event(enable_timing=True); c.record(stream)
        return a, b, c

    step(); torch.cuda.synchronize()
    k = max(1, min(args.steps, 3))
    marks = [step() for _ in range(k)]
    torch.cuda.synchronize()
    return {"steps": k, "h2d": h2d, "d2h": d2h,
            "comp_ms": sum(a.elapsed_time(b) for a, b, c in marks),
            "dec_ms": sum(b.elapsed_time(c) for a, b, c in marks),
            "total_ms": sum(a.elapsed_time(c) for a, b, c in marks)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="qp", choices=["qp", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--sequences", type=int, default=8,
                    help="independent sequences per GPU (their packed caches together exceed L2)")
    ap.add_argument("--seqs-per-call", type=int, default=4,
                    help="sequences whose layers go into one qp_decode_attn_layers call")
    ap.add_argument("--layers", type=int, default=0, help="profiling: keep only the first N layers of the workload")
    ap.add_argument("--batch", type=int, default=0, help="profiling: override the workload's batch size")
    ap.add_argument("--bits", type=int, default=0, choices=[0, 2, 4, 8, 16],
                    help="profiling: override the workload's code width (the token budget follows: tokens x bits constant)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-compress-layers", action="store_true", help="skip the qp_compress_layers figure")
    ap.add_argument("--no-generation", action="store_true", help="skip the append + decode generation-loop figure")
    ap.add_argument("--no-layer-chain", action="store_true", help="skip the layer-by-layer / CUDA-graph figures")
    ap.add_argument("--no-overlap", action="store_true", help="decode calls in plain stream order")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    args = ap.parse_args()
    wl = synth.WORKLOADS[args.workload]
    if args.layers or args.batch or args.bits:   # a variant of the same kernels, for ncu captures; never the bench line
        wl = synth.dataclasses.replace(wl, n_layers=args.layers or wl.n_layers, batch=args.batch or wl.batch,
                                       bits=args.bits or wl.bits,
                                       name=f"{wl.name}[layers={args.layers or wl.n_layers},batch={args.batch or wl.batch},"
                                            f"bits={args.bits or wl.bits}]")
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback "
                             "(use --impl reference for the CPU oracle)")
        run_gpu(args, wl)


if __name__ == "__main__":
    main()
