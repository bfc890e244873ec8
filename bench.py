#!/usr/bin/env python
"""Benchmark of the speculative semantic-ID decode step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b] [--mode 1] [--impl ours|reference]

One step = one nezha_decode call (draft head -> hash-set filter -> primary verify pass -> masked log-softmax /
beam top-k -> accept / roll back, all rounds) over the whole batch, always from the same prefilled state.
Prints ONE JSON line.  `value` = items (batch x beam) decoded per second with all inputs resident in HBM;
`e2e` = the same through the C ABI starting from pinned HOST histories (H2D copy + prefill + decode + D2H of
the results inside the timed region).  With N > 1 every rank runs an independent replica on its own GPU -- requests are
independent, so there is no collective on the data path -- and `value` sums the replicas (under torchrun, or started
by this script itself when it is called with --gpus N and no launcher).  The default workload is the largest
single-GPU configuration (the 7B shape); the default one-GPU run also times the other four configurations briefly and
reports them under `per_workload`.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

METRIC, UNIT = "items_per_s_decoded", "items/s"
# bumped whenever a kernel of the family changes in a way that can change its DRAM traffic: a traffic figure taken
# from an older revision is reported as null
KERNEL_REV = {"gemm": 7, "gemm_skinny": 2, "attention_tc": 3, "attention_umma": 5, "probe": 3}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, averaged over the launches of the class in one decode step
# (ncu, eager launches, L2 flushed before the step); key = class @ workload
NCU_TRAFFIC = {
    # captured on a two-layer cut of the 7B shape (the full model under ncu is a 68 s step); a launch is the same at any
    # depth, so the class average of the full model is rebuilt from the per-kernel figures: 12 layer launches per layer
    # (three rounds) moved 1,371 MB, the 16 launches outside the layers 436 MB -> (32 x 1,371 + 436) / 400
    "gemm@7b": {"family": "gemm", "kernel_rev": 7, "dram_bytes_per_launch": 110.8e6,
                "source": "profiles/gemm_tc_kernel_ncu.md, section E (two-layer cut, scaled by launches per layer)"},
    # the weight-streaming kernel, captured on a two-layer cut of the paper-shaped backbone (same widths): the four
    # projections of a layer read 8.61 + 67.25 + 34.02 + 12.75 MB, the LM-head rows 4.33 MB; a plain decode step of the
    # 16-layer model is 2 x (64 layer launches + 1) + 1 launches -> (2 x (16 x 122.63 + 4.33) + 2.1) / 131
    "gemm@paper": {"family": "gemm_skinny", "kernel_rev": 2, "dram_bytes_per_launch": 30.0e6,
                   "source": "profiles/gemm_skinny_kernel_ncu.md (two-layer cut, scaled by launches per layer)"},
    "gemm@small": {"family": "gemm", "kernel_rev": 6, "dram_bytes_per_launch": 3.18e6, "source": "profiles/gemm_tc_kernel_ncu.md, section A2"},
    "probe@0.5b@67108864": {"family": "probe", "kernel_rev": 3, "dram_bytes_per_launch": 5.10e9, "source": "profiles/hs_probe_kernel.md"},
    "attention@small": {"family": "attention_tc", "kernel_rev": 3, "dram_bytes_per_launch": 31.5e6,
                        "source": "profiles/attn_tc_kernel_ncu.md, traffic section"},
}


def ncu_traffic(key):
    rec = NCU_TRAFFIC.get(key)
    if rec and rec["kernel_rev"] == KERNEL_REV.get(rec["family"]):
        return rec
    return None


def whole_job_throughput(dist, local_ms: float, items_per_rank_step: int, steps: int, world: int, device="cpu"):
    """Replicas only: every rank decodes its own requests, nothing is exchanged on the data path.  The job's time is
    the slowest rank's (MAX over ranks of the device-timed region); its throughput counts the items of all ranks."""
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    if dist is not None and world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    worst_ms = float(t.item())
    return world * items_per_rank_step * steps / (worst_ms / 1e3), worst_ms


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU, sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def algorithmic_work(w, stats_tokens_per_step, rounds):
    """Algorithmic flops / bytes of one decode step, per kernel class.

    GEMM: 2 flops per (token, weight) pair of every projection and of the LM head rows of levels 2..L.
    Attention: the context K and V of every request once per (layer, pass) plus q and o of every token once
    (bytes); 4 * head_dim flops per (token, query head, visible position)."""
    esz = 4 if w.dtype == "fp32" else 2
    d, hd, Hq, Hkv, F, nl = w.d_model, w.head_dim, w.n_q_heads, w.n_kv_heads, w.d_ffn, w.n_layers
    per_tok_params = nl * ((Hq + 2 * Hkv) * hd * d + d * Hq * hd + 3 * F * d)
    lm = sum(w.T[1:]) * d
    gemm_flops = 2.0 * stats_tokens_per_step * (per_tok_params + lm)
    P = w.ctx_tokens
    # attention: the context KV of a request is read once per (request, layer, pass); queries and outputs once
    attn_bytes = rounds * nl * w.batch * (2 * Hkv * P * hd * esz) + stats_tokens_per_step * nl * 2 * Hq * hd * esz
    attn_flops = 4.0 * stats_tokens_per_step * nl * Hq * hd * (P + 2)
    # the weights of every projection (and of the LM head rows used) are read once per pass
    gemm_weight_bytes = rounds * (per_tok_params + lm) * esz
    return {"gemm_flops": gemm_flops, "attention_bytes": attn_bytes, "attention_flops": attn_flops,
            "gemm_weight_bytes": gemm_weight_bytes}


def probe_bench(args, w, eng, cat_dev, config, dev):
    """The hash-set probe alone: n keys (half catalogue items drawn at random, half uniform random tuples, shuffled),
    already packed and resident in HBM.  Algorithmic bytes per key: the 8-byte key, the 1-byte answer and one 32-byte
    bucket (at load factor 0.5 a probe sequence almost always ends in its first bucket)."""
    import torch
    n = args.probe_keys
    g = torch.Generator(device=dev); g.manual_seed(1234)
    half = n // 2
    idx = torch.randint(0, w.n_items, (half,), device=dev, generator=g)
    hits = cat_dev[idx]
    rnd = torch.stack([torch.randint(0, w.T[l], (n - half,), device=dev, generator=g, dtype=torch.int32) for l in range(w.L)], dim=1)
    codes = torch.cat([hits, rnd], dim=0)[torch.randperm(n, device=dev, generator=g)].contiguous()
    keys = eng.pack(codes)
    del codes, hits, rnd, idx
    found = torch.empty(n, dtype=torch.uint8, device=dev)
    for _ in range(max(args.warmup, 3)):
        eng.probe(keys, out=found)
    torch.cuda.synchronize()
    sampler = ClockSampler(int(dev.split(":")[1]))
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        eng.probe(keys, out=found)
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1) / args.steps
    peaks = load_peaks()
    gbs = n * 41.0 / (ms / 1e3) / 1e9
    rec = ncu_traffic(f"probe@{w.name}@{n}")
    traffic = rec["dram_bytes_per_launch"] if rec else None
    slots = 4 * max(2, math.ceil(math.ceil(max(1, w.n_items) / w.load_factor) / 4))      # buckets of four 8-byte slots
    print(json.dumps({"metric": "hash_probes_per_s", "value": n / (ms / 1e3), "unit": "probes/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "u64", "data": "synthetic",
                      "config": {"workload": config["workload"], "keys": n, "hit_fraction": float(found.float().mean()),
                                 "table_bytes": slots * 8, "l2": "keys alone (8 bytes each) exceed L2"},
                      "clocks": clocks, "gpu_launches": args.steps,
                      "roofline": {"kernel": "hs_probe_kernel", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"],
                                   "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": traffic,
                                   "of": peaks.get("source", "measured"),
                                   "algorithmic_bytes_per_key": 41}}))


def build_engine(w, dev, final_mask: str):
    """Weights, catalogue, histories and a prefilled engine for one workload; everything resident on the device."""
    import torch
    from paper_2511_18793_b200 import binding, synth
    weights = synth.make_weights(w, device=dev)
    catalog = synth.make_catalog(w)
    hist = synth.make_histories(w, catalog)
    cat_dev = torch.from_numpy(catalog).to(dev)
    eng = binding.Engine(binding.make_config(w), weights, cat_dev, w.load_factor, stream=torch.cuda.current_stream())
    n_unique = eng.build_hashset()
    assert n_unique == w.n_items
    eng.set_option(binding.OPT_FINAL_MASK, 1 if final_mask == "prefix" else 0)
    return {"w": w, "weights": weights, "catalog": catalog, "hist": hist, "cat_dev": cat_dev, "eng": eng}


def time_decode(ctx, mode, drafts, steps, warmup, flush, dist, world, dev, barrier, adaptive=False):
    """W warm-up steps, then K timed steps (one CUDA-event pair per step, L2 flushed before each, outside the events);
    then the per-class pass.  Returns the numbers of one workload."""
    import torch
    from paper_2511_18793_b200 import binding
    w, eng = ctx["w"], ctx["eng"]
    hist_pinned = torch.from_numpy(ctx["hist"]).pin_memory()
    nh_pinned = torch.full((w.batch,), w.n_hist, dtype=torch.int32).pin_memory()
    hist_dev = hist_pinned.to(dev, non_blocking=True)
    nh_dev = nh_pinned.to(dev, non_blocking=True)
    eng.prefill(hist_dev, nh_dev)
    eng.set_option(binding.OPT_ADAPTIVE_DRAFT, 1 if adaptive else 0)
    out = eng.alloc_outputs(w.batch, w.beam)
    items = w.batch * w.beam
    inject = None
    if drafts == "perfect" and mode == 1:
        art = eng.decode(w.beam, mode=2, trace=True)
        beams = art["trace"]["beams"].clone()
        inject = (beams, (beams[:, :, :, 0] >= 0).sum(dim=2).to(torch.int32).contiguous())

    def step():
        if inject is not None:
            return eng.decode_with_draft_tree(w.beam, inject[0], inject[1], out=out)
        return eng.decode(w.beam, mode=mode, out=out)

    for _ in range(warmup):
        flush.fill_(1)
        step()
    barrier()
    launches0 = binding.lib.nezha_launch_count()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    tokens = rounds = 0
    for a, b in evs:
        flush.fill_(1)
        a.record()
        r = step()
        b.record()
        tokens += r["stats"].primary_tokens
        rounds += r["stats"].rounds
    barrier()
    launches = binding.lib.nezha_launch_count() - launches0
    per_step_ms = [a.elapsed_time(b) for a, b in evs]
    value, total_ms_max = whole_job_throughput(dist, sum(per_step_ms), items, steps, world, dev)

    # ---- per-kernel-class CUDA-event timing (separate pass: two event records per launch perturb throughput)
    eng.profile_enable(True)
    eng.profile_read()
    prof_steps = max(3, min(steps, 10))
    ptok = prd = 0
    for _ in range(prof_steps):
        flush.fill_(1)
        r = step()
        ptok += r["stats"].primary_tokens
        prd += r["stats"].rounds
    prof = eng.profile_read()
    eng.profile_enable(False)
    peaks = load_peaks()
    work = algorithmic_work(w, ptok / prof_steps, prd / prof_steps)
    tot_prof_ms = sum(v["ms"] for v in prof.values()) or 1.0
    shares = {k: {"launches_per_step": v["launches"] / prof_steps, "ms_per_step": v["ms"] / prof_steps,
                  "share": v["ms"] / tot_prof_ms} for k, v in prof.items() if v["launches"]}
    dom = max(shares, key=lambda k: shares[k]["ms_per_step"])
    roof = {"kernel": dom, "bound": None, "achieved": None, "peak": None, "unit": None, "frac": None, "traffic": None,
            "of": peaks["source"]}
    dom_s = shares[dom]["ms_per_step"] / 1e3
    tf_peak, bw_peak = peaks["bf16_tflops_sustained"] * 1e12, peaks["hbm_gbs"] * 1e9
    if dom == "gemm" and w.dtype == "bf16" and work["gemm_weight_bytes"] / bw_peak > work["gemm_flops"] / tf_peak:
        # passes of a few rows: the projections are bound by reading every weight once per pass, not by flops
        ach = work["gemm_weight_bytes"] / dom_s / 1e9
        roof.update(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                    note="weight-streaming regime: weight bytes per pass / time of the GEMM class")
    elif dom == "gemm":
        ach = work["gemm_flops"] / dom_s / 1e12
        # fp32 workload: CUDA-core FMA peak = 148 SMs x 128 FMA lanes x 2 flops x 1.965 GHz = 74.4 TFLOP/s
        peak = peaks["bf16_tflops_sustained"] if w.dtype == "bf16" else 148 * 128 * 2 * 1.965e9 / 1e12
        roof.update(bound="tensor" if w.dtype == "bf16" else "alu", achieved=ach, peak=peak, unit="TFLOP/s", frac=ach / peak)
    elif dom == "attention":
        ach = work["attention_bytes"] / dom_s / 1e9
        roof.update(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
    else:
        roof.update(bound="latency", note="dominant class is neither GEMM nor attention")
    # DRAM traffic of the dominant kernel from the ncu capture of that kernel in this workload (bytes per launch);
    # null when no capture matches the current kernel revision
    rec = ncu_traffic(f"{dom}@{w.name}")
    if rec and rec["family"] == "gemm_skinny" and w.batch * w.beam * max(1, w.L - 1) > 128:
        rec = None                     # that capture is of the weight-streaming kernel: engines of at most 128 rows per pass
    if rec:
        roof["traffic"] = rec["dram_bytes_per_launch"]
        roof["traffic_source"] = rec["source"]
    if dom == "gemm":            # algorithmic bytes of an average launch of the class, to set beside `traffic`
        esz = 4 if w.dtype == "fp32" else 2
        act = (ptok / prof_steps) * (w.d_model * 4 + (w.n_q_heads + 2 * w.n_kv_heads) * w.head_dim + w.n_q_heads * w.head_dim
                                     + 3 * w.d_ffn) * esz * w.n_layers
        roof["algorithmic_bytes_per_launch"] = (work["gemm_weight_bytes"] + act) / max(1.0, shares["gemm"]["launches_per_step"])
    # the whole step against its floor: per class the larger of (bytes / copy bandwidth) and (flops / tensor peak),
    # summed over the GEMM and attention classes (the rest moves kilobytes), divided by the measured step time
    if w.dtype == "bf16" and mode != 0:
        tf, bw = peaks["bf16_tflops_sustained"] * 1e12, peaks["hbm_gbs"] * 1e9
        floor_s = max(work["gemm_flops"] / tf, work["gemm_weight_bytes"] / bw) + \
            max(work["attention_flops"] / tf, work["attention_bytes"] / bw)
        roof["step_floor_ms"] = floor_s * 1e3
        roof["step_frac"] = floor_s * 1e3 / (total_ms_max / steps)
    roof["classes"] = shares
    roof["attention_gbs"] = work["attention_bytes"] / (shares["attention"]["ms_per_step"] / 1e3) / 1e9 if "attention" in shares else None
    roof["attention_tflops"] = work["attention_flops"] / (shares["attention"]["ms_per_step"] / 1e3) / 1e12 if "attention" in shares else None
    roof["gemm_tflops"] = work["gemm_flops"] / (shares["gemm"]["ms_per_step"] / 1e3) / 1e12 if "gemm" in shares else None
    return {"value": value, "ms_per_step": total_ms_max / steps, "p50_ms": statistics.median(per_step_ms),
            "launches": int(launches), "rounds_per_step": rounds / steps, "primary_tokens_per_step": tokens / steps,
            "roofline": roof, "step": step, "out": out, "hist_pinned": hist_pinned, "nh_pinned": nh_pinned}


def workload_label(w):
    return (f"{w.name}: {w.n_layers}L d{w.d_model} {w.n_q_heads}q/{w.n_kv_heads}kv ffn{w.d_ffn}, "
            f"L={w.L} T={w.T[0]}, catalogue {w.n_items} ({w.catalog}), history {w.n_hist} items, "
            f"batch {w.batch} x beam {w.beam}, seed {w.seed}")


def reference_arm(args, w, config):
    """The CPU oracle as it stands on the host cores.  One step = the decode of ONE request of the workload (the first of
    the batch), from its prefilled state; the prefill is computed once before the loop and excluded, as in our arm."""
    import numpy as np
    from oracle import nezha_oracle as O
    from paper_2511_18793_b200 import synth
    weights = synth.make_weights(w, device="cpu")
    catalog = synth.make_catalog(w)
    hist = synth.make_histories(w, catalog, batch=1)
    Wn = synth.weights_to_numpy(weights)
    del weights
    shape = O.ModelShape(w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.d_ffn, w.L, tuple(w.T), w.rope_theta, w.rms_eps)
    big = w.d_model * w.d_ffn * w.n_layers > 2e8
    # multi-billion-parameter shapes: the oracle's fp32 arithmetic option (its fp64 default would convert 20 GB of weights
    # on every call); everything else as it stands
    odt = np.float32 if big else np.float64
    model = O.PrimaryModel(shape, Wn, cache_f64=not big, dtype=odt)
    head, valid = O.DraftHead(shape, Wn), O.ValidSet(catalog, w.T)
    req = model.prefill(hist[0])
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        if args.mode == 0:
            O.nezha_draft(head, req, w.beam, valid)
        elif args.mode == 2:
            O.ar_beam_search(model, req, w.beam, valid)
        else:
            O.speculative_decode(model, head, req, w.beam, valid)
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * sum(times) / len(times)
    v = w.beam / (ms / 1e3)
    try:
        import torch
        threads = torch.get_num_threads()
    except Exception:
        threads = os.cpu_count()
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                      "dtype": "f32" if big else "f64", "data": "synthetic", "config": config,
                      "cpu_baseline": {"value": v, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                       "sample": "decode of one request (the first of the batch, beam as configured) per "
                                                 "step; its prefill computed once before the loop and excluded",
                                       "blas_threads": threads},
                      "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def relaunch_replicas(args):
    """`--gpus N` without a launcher: start N replica processes, one per GPU, the way the launcher would."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="7b",
                    help="7b (default: the largest single-GPU configuration), 1.5b, 0.5b, small, tiny, paper")
    ap.add_argument("--mode", type=int, default=1, help="0 draft-only, 1 verified (default), 2 plain autoregressive")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--drafts", default="natural", choices=["natural", "perfect"],
                    help="mode 1 only: 'natural' = the (random-init) draft head's own draft tree; 'perfect' = the true beam "
                         "sets of every level injected as round 1's draft tree (best case: one round, everything accepted)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (requests per decode call)")
    ap.add_argument("--layers", type=int, default=0,
                    help="cut the backbone down to this many layers (profiler captures on a small case: a kernel's launch "
                         "is the same at any depth); the line then describes a cut-down workload, not the configuration")
    ap.add_argument("--items", type=int, default=0, help="cut the catalogue down to this many items (same purpose)")
    ap.add_argument("--final-mask", default="prefix", choices=["hash", "prefix"],
                    help="how the primary model's last-level validity mask (Eq. 5) is answered: the prefix map (the "
                         "library's default) or one hash-set probe per candidate code")
    ap.add_argument("--probe-keys", type=int, default=0,
                    help="instead of the decode step, time the stand-alone hash-set probe (Eq. 5) on this many keys, "
                         "half of them catalogue items, and print its own JSON line")
    ap.add_argument("--adaptive", action="store_true",
                    help="mode 1 with NEZHA_OPT_ADAPTIVE_DRAFT: a request stops drafting after a round that gained nothing "
                         "from its drafts (an engine policy; off by default, as in the library)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true",
                    help="skip the short runs of the other configurations that the default run adds under `per_workload`")
    ap.add_argument("--cpu-budget-s", type=float, default=20.0)
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        relaunch_replicas(args)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    import numpy as np
    import torch
    from paper_2511_18793_b200 import synth

    w = synth.WORKLOADS[args.workload]
    if args.batch > 0:
        w = synth.scaled(w, batch=args.batch)
    if args.layers > 0:
        w = synth.scaled(w, n_layers=args.layers)
    if args.items > 0:
        w = synth.scaled(w, n_items=args.items)
    config = {"workload": workload_label(w) + (" [cut down for profiling]" if args.layers > 0 or args.items > 0 else ""),
              "mode": {0: "draft-only (Algorithm 3)", 1: "verified (Algorithm 2)", 2: "autoregressive (Algorithm 1)"}[args.mode],
              "batch": w.batch, "beam": w.beam, "l2": "flushed between steps (256 MB write, outside the timed events)",
              "drafts": "natural (random-init draft head)" if args.drafts == "natural" or args.mode != 1 else
                        "perfect (the true beam sets injected as round 1's draft tree)"}

    # ------------------------------------------------------------------ reference arm: the oracle on host cores
    if args.impl == "reference":
        if rank == 0:
            reference_arm(args, w, config)
        return

    # ------------------------------------------------------------------ our arm
    from paper_2511_18793_b200 import binding
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=torch.device(dev))

    # a stream of its own (not the legacy default stream), so that the library may capture its rounds into CUDA graphs;
    # made current, so that the flushes, copies and timing events below are ordered on it too
    torch.cuda.set_stream(torch.cuda.Stream(device=dev))
    ctx = build_engine(w, dev, args.final_mask)
    eng = ctx["eng"]
    if args.probe_keys > 0:
        probe_bench(args, w, eng, ctx["cat_dev"], config, dev)
        return
    config["final_mask"] = "prefix map (one look-up per beam)" if args.final_mask == "prefix" else "hash-set probes"
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    items = w.batch * w.beam
    warmup = max(args.warmup, 3)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    res = time_decode(ctx, args.mode, args.drafts, args.steps, warmup, flush, dist, world, dev, barrier, adaptive=args.adaptive)
    if args.adaptive:
        config["drafts"] += ", drafting switched off per request after a round without gain"
    clocks = sampler.stop()
    step, out, hist_pinned, nh_pinned = res["step"], res["out"], res["hist_pinned"], res["nh_pinned"]

    # ---- end to end from pinned host memory: H2D histories, prefill, decode, D2H results
    host_codes = torch.empty(w.batch, w.beam, w.L, dtype=torch.int32).pin_memory()
    host_scores = torch.empty(w.batch, w.beam, dtype=torch.float32).pin_memory()
    host_count = torch.empty(w.batch, dtype=torch.int32).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        hd = hist_pinned.to(dev, non_blocking=True)
        nd = nh_pinned.to(dev, non_blocking=True)
        eng.prefill(hd, nd)
        step()
        host_codes.copy_(out["codes"], non_blocking=True)
        host_scores.copy_(out["scores"], non_blocking=True)
        host_count.copy_(out["count"], non_blocking=True)
        torch.cuda.synchronize()

    e2e_step()
    barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record()
    for _ in range(e2e_steps):
        e2e_step()
    eb.record()
    barrier()
    e2e_ms = max(ea.elapsed_time(eb), 0.0)
    e2e_value, e2e_ms_max = whole_job_throughput(dist, e2e_ms, items, e2e_steps, world, dev)
    h2d = hist_pinned.numel() * 4 + nh_pinned.numel() * 4
    d2h = host_codes.numel() * 4 + host_scores.numel() * 4 + host_count.numel() * 4

    line = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": res["ms_per_step"], "p50_ms": res["p50_ms"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic", "config": config,
            "clocks": clocks, "gpu_launches": res["launches"],
            "rounds_per_step": res["rounds_per_step"], "primary_tokens_per_step": res["primary_tokens_per_step"],
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "includes": "H2D histories + prefill + decode + D2H results", "steps": e2e_steps,
                    "ms_per_step": e2e_ms_max / e2e_steps},
            "roofline": res["roofline"]}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(ctx, args)

    # ---- the other configurations, briefly (one GPU, default run only): same step, fewer repetitions
    if world == 1 and not args.no_per_workload and args.workload == "7b" and args.batch == 0 and not args.layers and not args.items:
        per = {}
        del res, step, out
        ctx.clear(); eng.close(); del eng
        torch.cuda.empty_cache()
        for name in ("7b", "tiny", "small", "0.5b", "1.5b", "paper_batch1"):
            # (the last: the paper's own setting, one request at beam 10 -- passes of at most 20 rows, bound by the weights)
            wn = synth.scaled(synth.WORKLOADS["paper"], batch=1) if name == "paper_batch1" else synth.WORKLOADS[name]
            c2 = build_engine(wn, dev, args.final_mask)
            entry = {"workload": workload_label(wn)}
            for label, mode, drafts in (("verified", 1, "natural"), ("verified_adaptive", 1, "natural"),
                                        ("verified_perfect_tree", 1, "perfect"),
                                        ("autoregressive", 2, "natural"), ("draft_only", 0, "natural")):
                if name == "7b" and label == "verified" and args.mode == 1 and args.drafts == "natural" and not args.adaptive:
                    continue                                   # the headline of this line
                r2 = time_decode(c2, mode, drafts, 10, 3, flush, None, 1, dev, barrier, adaptive=label == "verified_adaptive")
                rf = r2["roofline"]
                entry[label] = {"value": r2["value"], "ms_per_step": r2["ms_per_step"], "p50_ms": r2["p50_ms"],
                                "rounds_per_step": r2["rounds_per_step"],
                                "primary_tokens_per_step": r2["primary_tokens_per_step"], "launches_per_step": r2["launches"] / 10,
                                "dominant": rf["kernel"], "bound": rf["bound"], "frac": rf["frac"],
                                "step_frac": rf.get("step_frac"), "gemm_tflops": rf.get("gemm_tflops"),
                                "attention_gbs": rf.get("attention_gbs")}
                del r2
            per[name] = entry
            c2["eng"].close(); c2.clear()
            torch.cuda.empty_cache()
        line["per_workload"] = per
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def cpu_baseline(ctx, args):
    """The oracle as it stands on the host cores, on a bounded sample of the same workload: the decode of its first
    request(s) until about `--cpu-budget-s` seconds of work (their prefill included) are done, at least one request; the
    prefill is excluded from the figure, as it is from ours."""
    import numpy as np
    import torch
    from oracle import nezha_oracle as O
    from paper_2511_18793_b200 import synth
    w = ctx["w"]
    Wn = synth.weights_to_numpy(ctx["weights"])
    shape = O.ModelShape(w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.d_ffn, w.L, tuple(w.T), w.rope_theta, w.rms_eps)
    big = w.d_model * w.d_ffn * w.n_layers > 2e8
    model = O.PrimaryModel(shape, Wn, cache_f64=not big, dtype=np.float32 if big else np.float64)
    head, valid = O.DraftHead(shape, Wn), O.ValidSet(ctx["catalog"], w.T)
    rows, t_decode, t_prefill = 0, 0.0, 0.0
    while rows < w.batch and t_decode + t_prefill < args.cpu_budget_s:
        t0 = time.perf_counter()
        req = model.prefill(ctx["hist"][rows])
        t1 = time.perf_counter()
        if args.mode == 0:
            O.nezha_draft(head, req, w.beam, valid)
        elif args.mode == 2:
            O.ar_beam_search(model, req, w.beam, valid)
        else:
            O.speculative_decode(model, head, req, w.beam, valid)
        t2 = time.perf_counter()
        t_prefill += t1 - t0
        t_decode += t2 - t1
        rows += 1
    return {"value": rows * w.beam / t_decode if t_decode > 0 else 0.0, "unit": UNIT, "cores": os.cpu_count(),
            "kind": "oracle", "blas_threads": torch.get_num_threads(),
            "arithmetic": "fp32 option of the oracle (multi-billion-parameter shape)" if big else "fp64",
            "sample": f"decode of the first {rows} request(s) of the batch ({t_decode:.1f} s; their prefill, "
                      f"{t_prefill:.1f} s, excluded)"}


if __name__ == "__main__":
    main()
