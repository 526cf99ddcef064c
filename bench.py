#!/usr/bin/env python
"""Benchmark of the quantized-pruning hot path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input: the
prefill-side compression (window scores -> top-k -> gather+quantize+pack) of every layer,
followed by every decode step's attention over the packed cache of every layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is the decode-attention throughput in GB/s of
algorithmic packed-cache bytes (codes + scale/zero) with everything resident in HBM; `e2e`
is the same byte count over a whole step whose inputs come from host memory and whose
results go back, through the same C-ABI calls.  The default workload is the largest
single-GPU configuration (Llama-3-70B shapes); `per_config` carries the decode figures of
the other configurations, each with one sequence per call.

With --gpus N > 1 and no WORLD_SIZE in the environment the script starts its own N ranks
(torch.distributed.run on 127.0.0.1), one GPU each; every rank runs its own sequences
(replicas, no data-path collective) and rank 0 prints the line.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2412_12706_b200 import shard, synth

METRIC = "decode_attn_hbm_gbs"
UNIT = "GB/s"
DEFAULT_WORKLOAD = synth.LLAMA70B_32K_B4.name
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126e6
DTYPE = "f16-mma/f32-acc"      # bf16 inputs and outputs, f16 tensor-core operands, f32 accumulation and softmax

# DRAM traffic of the decode attention kernel from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum per
# launch over the algorithmic bytes of that launch), valid only for the kernel sources they were taken on
# (sha256 of DECODE_KERNEL_SOURCES).  Captured on a few layers of the named workload; the traffic is proportional
# to the tiles streamed, so a full launch's traffic is ratio x its algorithmic bytes.
NCU_TRAFFIC: dict = {
    "sha256": "19c2c85de55d4ea6dd33aa50deecb688866ebceb1d17aca306556886ff7297c1",
    # (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes of the attention kernel's launch, mean of two
    # launches each: 16 layers x batch 1 of the 70B shapes (104.92 MB read + 5.05 MB written for 104.86 MB),
    # 3 layers of the 32k x batch-8 2-bit workload (151.29 + 3.62 for 150.99 MB), the 8k workload (84.18 + 2.74 for 83.89 MB)
    "ratio": {"llama3-70b-32k-b4-4bit-pyramid": 1.049, "llama3-8b-32k-b8-2bit": 1.026, "llama3-8b-8k-b1-4bit": 1.036},
}

KERNELS_PER_COMPRESS = 5      # sweep 1, sweep 2 (folds the row statistics), pool, top-k, gather+quantize (+ one 4-byte memset)
KERNELS_PER_DECODE_CALL = 2   # split-K attention, merge
DECODE_KERNEL_SOURCES = ("qp_decode.cu", "qp_decode_mma.cu", "qp_decode_mma2.cu", "qp_decode_mma8.cu",
                         "qp_decode_mma16.cu", "qp_mma.cuh")


def packed_bytes(wl: synth.Workload, layer: int) -> int:
    """Algorithmic bytes one decode step reads for one layer: codes plus fp16 scale and zero."""
    n, b, g = wl.n_keep(layer), wl.bits, wl.group
    elems = wl.batch * wl.n_kv_heads * n * wl.head_dim * 2            # K and V
    return elems * 2 if b == 16 else elems * (b + 32 // g) // 8


def model_bytes(wl: synth.Workload) -> int:
    return sum(packed_bytes(wl, l) for l in range(wl.n_layers))


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def decode_sources_sha() -> str:
    return hashlib.sha256(b"".join(open(os.path.join(ROOT, "paper_2412_12706_b200", "csrc", f), "rb").read()
                                   for f in DECODE_KERNEL_SOURCES)).hexdigest()


def ncu_traffic(name: str, bytes_per_call: float):
    if NCU_TRAFFIC.get("sha256") != decode_sources_sha():
        return None
    r = NCU_TRAFFIC["ratio"].get(name)
    return None if r is None else r * bytes_per_call


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
    """The CPU oracle, as it stands, on a bounded sample of the workload (sized for a few seconds of host
    time per step): the first layer(s) of one batch entry of one sequence, each compressed once and attended
    for `dec` decode steps."""
    from oracle import qp_oracle as orc
    u16 = synth.bits_u16
    dec = 8
    full_batch = wl.batch
    if wl.batch > 1:                                   # large configurations: one batch entry only
        wl = synth.dataclasses.replace(wl, batch=1)
    macs = wl.n_kv_heads * (wl.n_q_heads // wl.n_kv_heads) * wl.w * wl.L * wl.head_dim
    n_lay = max(1, min(wl.n_layers, 8, int(1e10 // macs)))
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
    units = wl.batch * wl.n_kv_heads                     # the oracle threads over (batch, KV head) only
    return {
        "decode_gbs": bytes_dec / statistics.mean(t_dec) / 1e9,
        "compress_tokens_per_s": wl.batch * wl.L / (statistics.mean(t_comp) / n_lay * wl.n_layers),
        "ms_per_step": 1e3 * (statistics.mean(t_comp) + statistics.mean(t_dec)),
        "cores": min(orc.num_threads(), units),
        "sample": f"layers 0..{n_lay - 1} of one sequence, batch entry 0 of {full_batch}: 1 compress_layer + {dec} "
                  f"decode steps per layer per step (of {wl.n_layers} layers x {wl.decode_steps} decode steps); "
                  f"compress tokens/s scaled to all {wl.n_layers} layers; {units} independent (batch, KV head) "
                  f"units, so at most {units} of the host's {orc.num_threads()} threads work",
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

def ev():
    return torch.cuda.Event(enable_timing=True)


def build_caches(qp, wl, seed, dev, ws_c, bits_list=None, keep_inputs=False):
    """Generates one sequence layer by layer from `seed`, compresses every layer at every code width of
    `bits_list` (default: the workload's own) and keeps only the packed caches unless keep_inputs.
    Returns ({bits: [Cache per layer]}, inputs or None, compress milliseconds per bits)."""
    bits_list = bits_list or [wl.bits]
    wls = synth.dataclasses.replace(wl, seed=seed)
    caches = {b: [] for b in bits_list}
    comp_ms = {b: 0.0 for b in bits_list}
    inputs = {"K": [], "V": [], "Qw": []} if keep_inputs else None
    stream = torch.cuda.current_stream()
    for l in range(wl.n_layers):
        k, v = synth.make_kv(wls, l, device=dev)
        qw = synth.make_q_win(wls, l, device=dev)
        for b in bits_list:
            wb = synth.dataclasses.replace(wls, bits=b)
            n = wb.n_keep(l)                        # buffers are allocated outside the timed call (an allocation can synchronise)
            c = qp.alloc_cache(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, b, wl.group, n, dev)
            kept = torch.empty((wl.batch, wl.n_kv_heads, n), dtype=torch.int32, device=dev)
            a, z = ev(), ev()
            a.record(stream)
            qp.compress_layer(k, v, qw, wb.layer_budget_bits(l), b, wl.group, wl.pool, c, kept, ws_c)
            z.record(stream)
            torch.cuda.synchronize()
            comp_ms[b] += a.elapsed_time(z)
            caches[b].append(c)
        if keep_inputs:
            inputs["K"].append(k); inputs["V"].append(v); inputs["Qw"].append(qw)
        del k, v, qw
    return caches, inputs, comp_ms


def time_calls(qp, batches, reps, overlap, stream):
    """Average duration of a qp_decode_attn_layers call over `reps` calls issued back to back, rotating over
    `batches` (consecutive calls touch different packed caches)."""
    qp.decode_overlap(overlap)
    for r in range(min(reps, 2 * len(batches) + 4)):
        qp.decode_attn_layers(batches[r % len(batches)])
    a, z = ev(), ev()
    a.record(stream)
    for r in range(reps):
        qp.decode_attn_layers(batches[r % len(batches)])
    z.record(stream)
    torch.cuda.synchronize()
    qp.decode_overlap(False)
    return a.elapsed_time(z) / reps


def per_config_figures(args, qp, dev, peak, stream, rank):
    """Decode figures of the other configurations of the contract, one sequence per call."""
    out = {}
    plans = [(synth.LLAMA8B_8K, None), (synth.LLAMA8B_32K_B8, None), (synth.sweep_128k(16), [16, 8, 4, 2])]
    for base, bits_list in plans:
        bits_list = bits_list or [base.bits]
        Bt, Hq, Hkv, D, L, w = base.batch, base.n_q_heads, base.n_kv_heads, base.head_dim, base.L, base.w
        ws_c = torch.empty(qp.compress_workspace_bytes(Bt, Hq, Hkv, D, L, w), dtype=torch.uint8, device=dev)
        smallest = min(model_bytes(synth.dataclasses.replace(base, bits=b)) for b in bits_list)
        n_rot = max(1, math.ceil(2.5 * L2_BYTES / smallest))     # rotate until consecutive launches cannot hit L2
        seqs, comp_ms = [], {b: 0.0 for b in bits_list}
        for s in range(n_rot):
            caches, _, cms = build_caches(qp, base, shard.sequence_seed(base.seed, rank, 64, s), dev, ws_c, bits_list)
            seqs.append(caches)
            for b in bits_list:
                comp_ms[b] += cms[b]
        for b in bits_list:
            wl = synth.dataclasses.replace(base, bits=b)
            name = base.name if len(bits_list) == 1 else synth.sweep_128k(b).name
            q = [[synth.make_q_dec(wl, l, t, device=dev) for l in range(wl.n_layers)] for t in range(4)]
            outs = [torch.empty_like(q[0][l]) for l in range(wl.n_layers)]
            ws_d = qp.new_decode_workspace(sum(qp.decode_workspace_bytes(c) for c in seqs[0][b]), dev)
            batches = [qp.LayerBatch(q[(i + s) % 4], seqs[s][b], outs, ws_d) for i in range(2) for s in range(n_rot)]
            bytes_call = model_bytes(wl)
            reps = int(max(32, min(4096, 0.08 / (bytes_call / 5e12))))     # about 0.1 s per figure: clocks settle under load
            ms_on = time_calls(qp, batches, reps, True, stream)
            ms_off = time_calls(qp, batches, reps, False, stream)
            ach = bytes_call / (ms_on * 1e-3) / 1e9
            out[name] = {
                "bits": b, "bytes_per_call": bytes_call, "sequences_rotated": n_rot, "calls_timed": reps,
                "us_per_call": ms_on * 1e3, "achieved": ach, "frac": ach / peak,
                "pct_of_nominal_8TBs": 100.0 * ach / NOMINAL_HBM_GBS,
                "stream_order_us_per_call": ms_off * 1e3,
                "stream_order_achieved": bytes_call / (ms_off * 1e-3) / 1e9,
                "traffic": ncu_traffic(name, bytes_call),
                "compress_ms_per_layer": comp_ms[b] / (n_rot * wl.n_layers),
                "compress_tokens_per_s": Bt * L / (comp_ms[b] * 1e-3 / n_rot),
            }
            del batches, ws_d
        del seqs, ws_c
        torch.cuda.empty_cache()
    return out


def strategy_figures(qp, dev, peak, stream, rank):
    """Decode figures of the rows beyond the main path, on the Llama-3-8B 8k shapes at 4 bit: the FlexGen arrangement
    (keys per token, g = 64, the paper's setting for it), outlier filtering (|x| > 6 kept in 16 bit) and head-level
    budgets.  One sequence per call where the entry point takes several caches."""
    wl = synth.LLAMA8B_8K
    Bt, Hq, Hkv, D, L, w = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.L, wl.w
    n, n_seq = wl.n_keep(0), 4
    ws_c = torch.empty(qp.compress_workspace_bytes(Bt, Hq, Hkv, D, L, w), dtype=torch.uint8, device=dev)
    flex, filt, heads = [], [], []
    st_flex = st_filt = None
    filt_cnt = 0
    for s in range(n_seq):
        wls = synth.dataclasses.replace(wl, seed=shard.sequence_seed(wl.seed, rank, 64, 32 + s))
        fl = []
        for l in range(wl.n_layers):
            k, v = synth.make_kv(wls, l, device=dev)
            qw = synth.make_q_win(wls, l, device=dev)
            _, kept = qp.compress_layer(k, v, qw, wl.budget_bits, 4, 32, wl.pool, workspace=ws_c)
            c = qp.alloc_cache(Bt, Hq, Hkv, D, 4, 64, n, dev)
            st_flex = st_flex or qp.make_strategy(c, 1, None)
            qp.gather_quantize_ex(k, v, kept, c, st_flex)
            fl.append(c)
            if s == 0 and l < 8:
                c2 = qp.alloc_cache(Bt, Hq, Hkv, D, 4, 32, n, dev)
                st2 = qp.make_strategy(c2, 0, 6.0)
                qp.gather_quantize_ex(k, v, kept, c2, st2)
                filt.append((c2, st2))
                heads.append(qp.compress_layer_heads(k, v, qw, n, 4, 32, wl.pool, k_axis=1))
        flex.append(fl)
    torch.cuda.synchronize()
    filt_cnt = sum(int(st.bufs[0][2].sum()) + int(st.bufs[1][2].sum()) for _, st in filt) / max(1, len(filt))
    qs = [synth.make_q_dec(wl, l, 0, device=dev) for l in range(wl.n_layers)]
    outs = [torch.empty_like(q) for q in qs]
    ws = qp.new_decode_workspace(sum(qp.decode_workspace_bytes(c) for c in flex[0]), dev)

    def timed(fn, reps):
        for _ in range(3):
            fn(0)
        a, z = ev(), ev()
        a.record(stream)
        for r in range(reps):
            fn(r)
        z.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(z) / reps

    flex_bytes = Bt * Hkv * n * D * 2 * (4 + 32 // 64) // 8 * wl.n_layers
    ms = timed(lambda r: qp.decode_attn_layers_ex(qs, flex[r % n_seq], st_flex, outs, ws), 512)
    layer_bytes = Bt * Hkv * n * D * 2 * (4 + 1) // 8
    ms_f = timed(lambda r: qp.decode_attn_ex(qs[0], filt[r % len(filt)][0], filt[r % len(filt)][1], outs[0], ws), 64)
    G = Hq // Hkv
    hq = [qs[0].view(Bt * Hkv, 1, G, D)[i] for i in range(Bt * Hkv)]          # per-head views, built once
    ho = [outs[0].view(Bt * Hkv, 1, G, D)[i] for i in range(Bt * Hkv)]
    ms_h = timed(lambda r: qp.decode_attn_layers_ex(hq, heads[r % len(heads)].caches, heads[r % len(heads)].strategy, ho, ws), 64)
    head_tokens = sum(sum(h.n_heads) for h in heads) / len(heads)
    return {
        "workload": wl.name + ", 4 bit",
        "flexgen_g64": {"note": "keys and values per token, group 64; qp_decode_attn_layers_ex, 32 layers per call, plain "
                                "stream order, rotating over 4 sequences", "bytes_per_call": flex_bytes,
                        "us_per_call": ms * 1e3, "achieved": flex_bytes / (ms * 1e-3) / 1e9,
                        "frac": flex_bytes / (ms * 1e-3) / 1e9 / peak},
        "kivi_outliers": {"note": "per-channel keys, |x| > 6 kept in 16 bit (side lists); qp_decode_attn_ex, one layer per "
                                  "call (the chunked kernel)", "outliers_per_layer": filt_cnt,
                          "us_per_layer_call": ms_f * 1e3, "GB/s": layer_bytes / (ms_f * 1e-3) / 1e9},
        "head_budgets": {"note": "per-head token counts under a shared layer budget, keys per token; one layer per call "
                                 "(8 per-head caches in one qp_decode_attn_layers_ex call)",
                         "tokens_per_head_min_max": [min(min(h.n_heads) for h in heads), max(max(h.n_heads) for h in heads)],
                         "us_per_layer_call": ms_h * 1e3,
                         "GB/s": head_tokens * D * 2 * (4 + 1) / 8 / (ms_h * 1e-3) / 1e9},
    }


def run_gpu(args, wl):
    from paper_2412_12706_b200 import qp
    dist, rank, world, local = shard.init_ranks("nccl")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    qp.lib()
    peak, peak_kind = hbm_peak()

    n_layers, n_dec = wl.n_layers, wl.decode_steps
    bytes_seq = model_bytes(wl)
    # sequences per GPU: enough packed cache that consecutive launches cannot be served from L2
    n_seq = args.sequences or max(1, math.ceil(2.5 * L2_BYTES / bytes_seq))
    per_call = max(1, min(args.seqs_per_call, n_seq, qp.QP_MAX_LAYERS // n_layers))
    while n_seq % per_call:
        per_call -= 1
    Bt, Hq, Hkv, D, L, w = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.L, wl.w
    stream = torch.cuda.current_stream()
    overlap = not args.no_overlap

    # ---- inputs resident in HBM: every rank and every sequence has its own seed
    ws_c = torch.empty(qp.compress_workspace_bytes(Bt, Hq, Hkv, D, L, w), dtype=torch.uint8, device=dev)
    seqs = []
    for s in range(n_seq):
        seed = shard.sequence_seed(wl.seed, rank, n_seq, s)
        caches, inputs, _ = build_caches(qp, wl, seed, dev, ws_c, keep_inputs=True)
        wls = synth.dataclasses.replace(wl, seed=seed)
        n_q = min(n_dec, 8)                                  # distinct query sets, reused cyclically over the decode steps
        qdec = torch.stack([torch.stack([synth.make_q_dec(wls, l, t, device=dev) for l in range(n_layers)])
                            for t in range(n_q)])            # [n_q, n_layers, Bt, Hq, D]
        sq = {"K": inputs["K"], "V": inputs["V"], "Qw": inputs["Qw"], "qdec": qdec, "cache": caches[wl.bits], "seed": seed}
        sq["kept"] = [torch.empty((Bt, Hkv, wl.n_keep(l)), dtype=torch.int32, device=dev) for l in range(n_layers)]
        sq["out"] = torch.empty((n_layers, Bt, Hq, D), dtype=torch.bfloat16, device=dev)
        sq["ws_bytes"] = sum(qp.decode_workspace_bytes(c) for c in sq["cache"])
        seqs.append(sq)
    groups = []
    for g0 in range(0, n_seq, per_call):
        members = seqs[g0:g0 + per_call]
        ws_g = qp.new_decode_workspace(sum(m["ws_bytes"] for m in members), dev)
        groups.append([qp.LayerBatch([m["qdec"][t, l] for m in members for l in range(n_layers)],
                                     [c for m in members for c in m["cache"]],
                                     [m["out"][l] for m in members for l in range(n_layers)], ws_g)
                       for t in range(seqs[0]["qdec"].shape[0])])
    n_q = seqs[0]["qdec"].shape[0]

    dec_bytes_step = n_seq * n_dec * bytes_seq
    dec_bytes_call = per_call * bytes_seq
    ctx_tokens_step = n_seq * Bt * L
    input_bytes = 2 * n_seq * n_layers * Bt * Hkv * L * D * 2

    def compress_all():
        for sq in seqs:
            for l in range(n_layers):
                qp.compress_layer(sq["K"][l], sq["V"][l], sq["Qw"][l], wl.layer_budget_bits(l), wl.bits, wl.group,
                                  wl.pool, sq["cache"][l], sq["kept"][l], ws_c)

    def decode_all():
        # no event between the calls: with the overlap enabled consecutive decode calls share the GPU (the next
        # call's attention kernel starts while this call's merge step runs), and an event record would forbid that
        for t in range(n_dec):
            for grp in groups:       # consecutive launches touch different sequences' caches
                qp.decode_attn_layers(grp[t % n_q])
    n_calls_step = n_dec * len(groups)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    qp.decode_overlap(overlap)       # the decode steps are independent and nothing else is enqueued between them
    for _ in range(args.warmup):
        compress_all(); decode_all()
    barrier()

    sampler = ClockSampler(local) if rank == 0 else None
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
    qp.decode_overlap(False)

    total_ms = t_begin.elapsed_time(t_end)
    comp_ms = sum(a.elapsed_time(b) for a, b, c in marks)
    dec_ms = sum(b.elapsed_time(c) for a, b, c in marks)
    call_ms = dec_ms / (args.steps * n_calls_step)      # average launch duration over the timed decode phases

    extras = {}
    if not args.lean and world == 1:       # single-GPU side figures
        # ---- the same decode calls in plain stream order (the library's default), compared fairly: the SM clock under
        # the power cap moves with the load of the last few hundred milliseconds, so the two orders alternate in
        # segments inside one sustained loop (a short loop after an idle moment runs at a higher clock than the
        # timed region and flatters whatever it times)
        flat = [grp[t] for t in range(n_q) for grp in groups]
        seg = int(max(16, min(1024, 0.1 / (dec_bytes_call / 5e12))))
        on_ms, off_ms = [], []
        for rnd in range(4):
            on_ms.append(time_calls(qp, flat, seg, True, stream))
            off_ms.append(time_calls(qp, flat, seg, False, stream))
        on_ms, off_ms = on_ms[1:], off_ms[1:]                    # the first round brings the clock down
        off, on = sum(off_ms) / len(off_ms), sum(on_ms) / len(on_ms)
        extras["decode_stream_order"] = {
            "note": "the same calls without qp_decode_overlap (the library's default); overlap and plain order "
                    f"alternate in segments of {seg} calls inside one sustained loop, first round dropped",
            "us_per_call": off * 1e3, "GB/s": dec_bytes_call / (off * 1e-3) / 1e9,
            "overlap_us_per_call_same_loop": on * 1e3, "overlap_GB/s_same_loop": dec_bytes_call / (on * 1e-3) / 1e9}

        # ---- compression with all layers of a sequence in one qp_compress_layers call
        if Bt * n_layers * Hkv <= 65535 and qp.compress_workspace_bytes(Bt * n_layers, Hq, Hkv, D, L, w) < 24e9:
            ws_cl = torch.empty(qp.compress_workspace_bytes(Bt * n_layers, Hq, Hkv, D, L, w), dtype=torch.uint8, device=dev)
            budgets = [wl.layer_budget_bits(l) for l in range(n_layers)]

            def compress_all_layers():
                for sq in seqs:
                    qp.compress_layers(sq["K"], sq["V"], sq["Qw"], budgets, wl.bits, wl.group, wl.pool, sq["cache"],
                                       sq["kept"], ws_cl)
            compress_all_layers()
            k0, k1 = ev(), ev()
            k0.record(stream)
            for _ in range(3):
                compress_all_layers()
            k1.record(stream)
            torch.cuda.synchronize()
            cl_ms = k0.elapsed_time(k1) / 3
            extras["compress_layers_call"] = {
                "note": f"qp_compress_layers: the {n_layers} layers of a sequence per call, one launch per stage",
                "ms_per_layer": cl_ms / (n_seq * n_layers), "tokens_per_s": world * ctx_tokens_step / (cl_ms * 1e-3)}
            del ws_cl

        # ---- layer by layer: one qp_decode_attn call per layer in plain stream order (what a model's decode loop
        #      does between its other kernels), issued from Python and replayed from a CUDA graph
        sq0 = seqs[0]
        qs0, outs0 = sq0["qdec"][0], sq0["out"]
        ws_l = qp.new_decode_workspace(max(qp.decode_workspace_bytes(c) for c in sq0["cache"]), dev)

        def chain():
            for l in range(n_layers):
                qp.decode_attn(qs0[l], sq0["cache"][l], outs0[l], ws_l)
        for _ in range(3):
            chain()
        reps = 8
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
        extras["decode_layer_by_layer"] = {
            "note": "one sequence, one qp_decode_attn call per layer, plain stream order",
            "us_per_layer_call": layer_ms * 1e3 / n_layers, "GB/s": bytes_seq / (layer_ms * 1e-3) / 1e9,
            "cuda_graph_us_per_layer_call": graph_ms * 1e3 / n_layers,
            "cuda_graph_GB/s": bytes_seq / (graph_ms * 1e-3) / 1e9}
        del graph, ws_l

        # ---- generation loop: every decode step first appends the new token's key/value rows to every layer
        #      (qp_append_kv_layers; full tails are quantized into the caches) and then attends over packed
        #      tokens plus tail (qp_decode_attn_tail_layers).  Same grouping of sequences per call as above.
        g_steps = 2 * wl.group + 8 if wl.bits < 16 else 72      # two flushes of every tail on the way
        room = 3 * wl.group if wl.bits < 16 else g_steps + 8
        gen_groups = []
        for g0_ in range(0, n_seq, per_call):
            members = seqs[g0_:g0_ + per_call]
            caches, tails, kn, vn = [], [], [], []
            for m in members:
                wls = synth.dataclasses.replace(wl, seed=m["seed"])
                for l in range(n_layers):
                    c, _ = qp.compress_layer(m["K"][l], m["V"][l], m["Qw"][l], wl.layer_budget_bits(l), wl.bits,
                                             wl.group, wl.pool, workspace=ws_c, n_cap=wl.n_keep(l) + room)
                    caches.append(c); tails.append(qp.alloc_tail(c))
                    a, b_ = synth.make_kv_new(wls, l, 0, device=dev)
                    kn.append(a); vn.append(b_)
            gen_groups.append(qp.GenBatch([m["qdec"][0, l] for m in members for l in range(n_layers)], kn, vn, caches,
                                          tails, [m["out"][l] for m in members for l in range(n_layers)]))
        gen_tok0 = sum(gb.cache_arr[i].n_keep for gb in gen_groups for i in range(gb.n))

        def gen_step():
            for gb in gen_groups:
                qp.append_kv_layers(gb)
                qp.decode_attn_tail_layers(gb)
        qp.decode_overlap(overlap)
        for _ in range(4):
            gen_step()
        e0, e1 = ev(), ev()
        e0.record(stream)
        for _ in range(g_steps - 4):
            gen_step()
        e1.record(stream)
        torch.cuda.synchronize()
        qp.decode_overlap(False)
        gen_ms = e0.elapsed_time(e1) / ((g_steps - 4) * len(gen_groups))
        gen_tok1 = sum(gb.cache_arr[i].n_keep for gb in gen_groups for i in range(gb.n))
        # packed bytes a call reads, averaged over the loop (the caches grow by a group at every flush)
        per_tok = Bt * Hkv * D * 2 * (2.0 if wl.bits == 16 else (wl.bits + 32 // wl.group) / 8)
        gen_call_bytes = 0.5 * (gen_tok0 + gen_tok1) * per_tok / len(gen_groups)
        extras["decode_with_append"] = {
            "note": "per decode step and group of sequences: qp_append_kv_layers (new rows into the bf16 tails; "
                    "full tails quantized into the caches) + qp_decode_attn_tail_layers (packed tokens + tail)",
            "steps": g_steps - 4, "us_per_step_call": gen_ms * 1e3, "GB/s": gen_call_bytes / (gen_ms * 1e-3) / 1e9,
            "launches_per_step_call": "3 (4 on the steps that flush)"}
        del gen_groups

    # ---- end to end: host buffers in, host buffers out, through the same calls
    e2e = None if args.no_e2e else run_e2e(args, wl, qp, seqs, groups, ws_c, dev, stream, per_call)

    # ---- the other configurations (decode, one sequence per call); the main workload's inputs are released first
    per_config = strategies = None
    if not args.no_per_config and world == 1:
        for sq in seqs:
            sq["K"].clear(); sq["V"].clear(); sq["Qw"].clear()
        torch.cuda.empty_cache()
        per_config = per_config_figures(args, qp, dev, peak, stream, rank)
        strategies = strategy_figures(qp, dev, peak, stream, rank)
    barrier()

    def allmax(x: float) -> float:
        return shard.max_over_ranks(x, dist, dev)

    total_ms, comp_ms, dec_ms = allmax(total_ms), allmax(comp_ms), allmax(dec_ms)
    e2e_ms = allmax(e2e["total_ms"]) if e2e else None
    if rank != 0:
        shard.finish_ranks(dist)
        return

    steps = args.steps
    value = shard.whole_job_throughput(dec_bytes_step * steps, world, dec_ms * 1e-3) / 1e9
    achieved = dec_bytes_call / (call_ms * 1e-3) / 1e9
    cpu = oracle_sample(wl, 1, 0) if world == 1 and not args.no_cpu_baseline else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": args.warmup,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": wl.name, "layers": n_layers, "batch": Bt, "q_heads": Hq, "kv_heads": Hkv,
                   "head_dim": D, "context": L, "window": w, "bits": wl.bits, "group": wl.group,
                   "n_keep": [wl.n_keep(0), wl.n_keep(n_layers - 1)], "decode_steps": n_dec,
                   "sequences_per_gpu": n_seq, "parallelism": f"replicas x{world}, no collective",
                   "decode_api": f"qp_decode_attn_layers: one launch pair per decode step over all {n_layers} layers of "
                                 f"{per_call} sequence(s) ({dec_bytes_call / 1e6:.0f} MB per call)",
                   "sequences_per_call": per_call,
                   "call_overlap": overlap,
                   "l2": f"inputs larger than L2: a decode step reads {n_seq * bytes_seq / 1e6:.0f} MB of packed cache "
                         f"({n_seq} sequence(s), consecutive launches read different data); compress inputs "
                         f"{input_bytes / 1e9:.2f} GB"},
        "compress_tokens_per_s": world * ctx_tokens_step * steps / (comp_ms * 1e-3),
        "compress_ms_per_layer": comp_ms / (steps * n_seq * n_layers),
        "decode_us_per_call": call_ms * 1e3,
        "decode_phase_ms_per_step": dec_ms / steps,
        "pct_of_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "kernel": "decode attention (split-K attention kernel + merge kernel, per call)",
                     "achieved": achieved,
                     "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                     "traffic": ncu_traffic(wl.name, dec_bytes_call)},
        "e2e": None if e2e is None else {
            "value": world * dec_bytes_step * e2e["steps"] / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
            "note": "decode bytes of a step over the WHOLE step (uploads, compression, decode, downloads); " + e2e["note"],
            "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
            "ms_per_step": e2e["total_ms"] / e2e["steps"],
            "decode_phase_GB/s": dec_bytes_step * e2e["steps"] / (e2e["dec_ms"] * 1e-3) / 1e9,
            "compress_tokens_per_s": world * ctx_tokens_step * e2e["steps"] / (e2e["comp_ms"] * 1e-3)},
        "gpu_launches": steps * (n_seq * n_layers * KERNELS_PER_COMPRESS + n_calls_step * KERNELS_PER_DECODE_CALL),
        "clocks": clocks,
        "per_config": per_config,
        "strategies": strategies,
    }
    line.update(extras)
    if cpu is not None:
        line["cpu_baseline"] = {"value": cpu["decode_gbs"], "unit": UNIT, "cores": cpu["cores"], "kind": "oracle",
                                "sample": cpu["sample"], "compress_tokens_per_s": cpu["compress_tokens_per_s"]}
    print(json.dumps(line))
    shard.finish_ranks(dist)


def run_e2e(args, wl, qp, seqs, groups, ws_c, dev, stream, per_call):
    """The same step with every input starting in host memory and every decode output read back.  K, V and
    Q_win of a layer are staged through two reused pinned buffers (the host copy of all inputs is ordinary
    memory, it would be too large to pin) and uploaded before that layer's qp_compress_layer; each decode step
    uploads its queries from pinned memory and downloads its outputs into pinned memory."""
    n_layers, n_dec = wl.n_layers, wl.decode_steps
    layer_bytes = seqs[0]["K"][0].numel() * 2
    try:
        import psutil
        avail = psutil.virtual_memory().available
    except Exception:
        avail = 32e9
    total_layers = len(seqs) * n_layers
    held = int(max(1, min(total_layers, (0.45 * avail) // (2 * layer_bytes))))
    # host copies (pageable) of the first `held` layers' K and V; further layers reuse them cyclically
    flat = [(sq, l) for sq in seqs for l in range(n_layers)]
    hK = [flat[i][0]["K"][flat[i][1]].cpu() for i in range(held)]
    hV = [flat[i][0]["V"][flat[i][1]].cpu() for i in range(held)]
    hQ = [sq["Qw"][l].cpu().pin_memory() for sq, l in flat]
    pin = [(torch.empty_like(hK[0]).pin_memory(), torch.empty_like(hV[0]).pin_memory()) for _ in range(2)]
    pin_free = [ev() for _ in range(2)]
    dK, dV = torch.empty_like(seqs[0]["K"][0]), torch.empty_like(seqs[0]["V"][0])
    dQ = torch.empty_like(seqs[0]["Qw"][0])
    n_q = seqs[0]["qdec"].shape[0]
    egroups = []
    for gi, g0 in enumerate(range(0, len(seqs), per_call)):
        ids = list(range(g0, g0 + per_call))
        hq_g = torch.stack([seqs[i]["qdec"] for i in ids], dim=1).cpu().pin_memory()     # [n_q, per_call, layers, Bt, Hq, D]
        dq_g = torch.empty_like(hq_g[0], device=dev)
        dout_g = torch.empty_like(dq_g)
        hout_g = torch.empty_like(hq_g[0]).pin_memory()
        batch = qp.LayerBatch([dq_g[j, l] for j in range(per_call) for l in range(n_layers)],
                              [c for i in ids for c in seqs[i]["cache"]],
                              [dout_g[j, l] for j in range(per_call) for l in range(n_layers)], groups[gi][0].workspace)
        egroups.append((hq_g, dq_g, dout_g, hout_g, batch))
    h2d = total_layers * (2 * layer_bytes + hQ[0].numel() * 2) + n_dec * sum(g[1].numel() * 2 for g in egroups)
    d2h = n_dec * sum(g[2].numel() * 2 for g in egroups)

    def step():
        a = ev(); a.record(stream)
        for i, (sq, l) in enumerate(flat):
            pk, pv = pin[i % 2]
            if i >= 2:
                pin_free[i % 2].synchronize()                       # the upload that last used this buffer is done
            pk.copy_(hK[i % held]); pv.copy_(hV[i % held])
            dK.copy_(pk, non_blocking=True); dV.copy_(pv, non_blocking=True)
            pin_free[i % 2].record(stream)
            dQ.copy_(hQ[i], non_blocking=True)
            qp.compress_layer(dK, dV, dQ, wl.layer_budget_bits(l), wl.bits, wl.group, wl.pool,
                              sq["cache"][l], sq["kept"][l], ws_c)
        b = ev(); b.record(stream)
        for t in range(n_dec):
            for hq_g, dq_g, dout_g, hout_g, batch in egroups:
                dq_g.copy_(hq_g[t % n_q], non_blocking=True)
                qp.decode_attn_layers(batch)
                hout_g.copy_(dout_g, non_blocking=True)
        c = ev(); c.record(stream)
        return a, b, c

    step(); torch.cuda.synchronize()
    k = max(1, min(args.steps, 2))
    marks = []
    for _ in range(k):
        marks.append(step())
        torch.cuda.synchronize()
    note = (f"K/V of every layer copied from ordinary host memory into one of two pinned staging buffers and uploaded "
            f"from there ({2 * layer_bytes / 1e6:.0f} MB per layer)")
    if held < total_layers:
        note += f"; the host holds {held} of {total_layers} layers' K/V and reuses them cyclically"
    return {"steps": k, "h2d": h2d, "d2h": d2h, "note": note,
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
    ap.add_argument("--sequences", type=int, default=0,
                    help="independent sequences per GPU (default: as many as make the packed caches exceed L2)")
    ap.add_argument("--seqs-per-call", type=int, default=1,
                    help="sequences whose layers go into one qp_decode_attn_layers call (default 1: the configuration's own batch)")
    ap.add_argument("--layers", type=int, default=0, help="profiling: keep only the first N layers of the workload")
    ap.add_argument("--batch", type=int, default=0, help="profiling: override the workload's batch size")
    ap.add_argument("--bits", type=int, default=0, choices=[0, 2, 4, 8, 16],
                    help="profiling: override the workload's code width (the token budget follows: tokens x bits constant)")
    ap.add_argument("--decode-steps", type=int, default=0, help="profiling: override the number of decode steps")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap", action="store_true", help="decode calls in plain stream order in the timed region too")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-per-config", action="store_true", help="skip the other configurations' decode figures")
    ap.add_argument("--lean", action="store_true",
                    help="profiling: only the timed region (no side figures: stream-order calls, layer chain, generation loop)")
    args = ap.parse_args()
    wl = synth.WORKLOADS[args.workload]
    if args.layers or args.batch or args.bits or args.decode_steps:   # a cut-down variant for ncu captures; never the bench line
        wl = synth.dataclasses.replace(wl, n_layers=args.layers or wl.n_layers, batch=args.batch or wl.batch,
                                       bits=args.bits or wl.bits, decode_steps=args.decode_steps or wl.decode_steps,
                                       name=f"{wl.name}[layers={args.layers or wl.n_layers},batch={args.batch or wl.batch},"
                                            f"bits={args.bits or wl.bits}]")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(shard.spawn_ranks(args.gpus, [os.path.abspath(__file__)] + sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback "
                             "(use --impl reference for the CPU oracle)")
        run_gpu(args, wl)


if __name__ == "__main__":
    main()
