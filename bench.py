#!/usr/bin/env python
"""Benchmark of the token-tree verification pass (one step = one whole pass: mask table, decoder
forward over all tree nodes, argmax, verified-path search, cache rollback).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2|C3|C5|C1] [--impl reference]

Prints ONE JSON line. The path does not shard (one GPU per model replica, no collective): with
--gpus N > 1, launched under torchrun, every rank runs an independent replica of the same
workload and the value is the replicas' total.

What the line holds (GPU arm):
  value / ms_per_step     median of the K per-step times (CUDA events between the steps, no host
                          synchronisation inside the timed region), max over ranks; min, max and mean beside it
  roofline                the dominant kernel (the weight-streaming GEMM) INSIDE an undisturbed pass: a second
                          region of K passes records %globaltimer stamps per launch (llmcad_set_gemm_trace);
                          a launch is charged the time from the end of its predecessor to its own end, so the
                          kernels' times add up to the pass; `isolated` is the same kernel bracketed by events
                          (which switches off the overlap of consecutive launches)
  e2e                     the same pass through the host-buffer entry point, logits included
  workloads               the 13B configuration (C3) timed in the same process, and a digest of the
                          attention-only sweep (C4); only with the default workload on one GPU
  cpu_baseline            the CPU oracle, as it stands, on this machine's host cores
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2309_04255_b200 import inputs as gen  # noqa: E402

METRIC = "tree_verification_passes_per_sec"
UNIT = "passes/s"
# DRAM traffic of one GEMM (streaming + finishing kernel) from the ncu capture named here (dram__bytes_read.sum +
# dram__bytes_write.sum of both kernels, caches flushed between them) next to its algorithmic bytes; the traffic is the
# weight stream, which grows in proportion to the bytes, so other GEMMs are scaled by the ratio.
NCU_GEMM_CAPTURE = {"summary": "profiles/gemm_stream_kernel__7b_qkv_n32.md", "dram_bytes": 108.45e6, "algorithmic_bytes": 102.5e6}


def algorithmic_bytes(cfg, P, n, int4=False):
    """Bytes one pass must move: every weight matrix once, the prefix K/V once, the tree nodes'
    K/V written and read once, the embedding rows of the n tokens, the fp32 logits. With INT4 weights
    the layer matrices take half a byte per element plus one exponent byte per group of 64."""
    e = cfg.elem_bytes
    weights = cfg.weight_bytes()
    if int4:
        weights = int(cfg.n_layers * cfg.layer_weight_elems() * (0.5 + 1.0 / 64)) + cfg.vocab * cfg.d_model * e
    prefix_kv = 2 * cfg.n_layers * P * cfg.d_model * e
    tree_kv = 2 * 2 * cfg.n_layers * n * cfg.d_model * e
    logits = n * cfg.vocab * 4
    embed = n * cfg.d_model * e
    return {"weights": weights, "prefix_kv": prefix_kv, "tree_kv": tree_kv, "logits": logits, "embed": embed,
            "total": weights + prefix_kv + tree_kv + logits + embed}


def gemm_algorithmic_bytes(cfg, n):
    """Summed over the GEMM launches of one pass: the weight matrix, its bf16 input rows and
    its outputs (q/k/v rows, fp32 residual read+write, SwiGLU rows, fp32 logits)."""
    d, f, v, e = cfg.d_model, cfg.d_ffn, cfg.vocab, cfg.elem_bytes
    per_layer = (3 * d * d + d * d + 2 * f * d + d * f) * e           # weights
    per_layer += n * (d + d + d + f) * e                              # inputs of the four GEMMs
    per_layer += n * (3 * d * e + 2 * d * 4 + f * e + 2 * d * 4)      # outputs
    head = v * d * e + n * d * e + n * v * 4
    return cfg.n_layers * per_layer + head, cfg.n_layers * 4 + 1


def flops(cfg, P, n):
    d, f, v = cfg.d_model, cfg.d_ffn, cfg.vocab
    per_layer = 2 * n * (4 * d * d + 3 * d * f) + 4 * n * (P + n) * d
    return cfg.n_layers * per_layer + 2 * n * v * d


class ClockSampler:
    """SM clock, power and throttle reasons read through NVML every few milliseconds by a thread of this
    process (reading only; nothing is set). `mark()` opens and closes named windows, so that the samples
    taken during the timed region can be told from the rest."""
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples, self.windows, self.period = [], {}, period_s
        self.h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:   # no NVML: the line says so
            self.err = repr(e)
        self._stop = threading.Event()
        self.t = threading.Thread(target=self._run, daemon=True)
        if self.h is not None:
            self.t.start()

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append((time.perf_counter(), float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)),
                                     nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0,
                                     int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))))
            except Exception:
                pass
            self._stop.wait(self.period)

    def mark(self, name, t0, t1):
        self.windows[name] = (t0, t1)

    def settle(self, limit_s: float = 4.0) -> float:
        """Waits (idle, at most limit_s) until the power or thermal reason that the set-up of a workload may have left
        behind (generating and packing tens of GB of weights draws close to the power limit) is no longer reported,
        so that the timed region starts from the clocks the pass itself sustains. Returns the seconds waited."""
        if self.h is None:
            return 0.0
        t0 = time.perf_counter()
        mask = 0
        for b in self.REASONS.values():
            mask |= b
        while time.perf_counter() - t0 < limit_s:
            recent = self.samples[-8:]
            if len(recent) >= 8 and not any(smp[3] & mask for smp in recent):
                break
            time.sleep(0.05)
        return time.perf_counter() - t0

    def stop(self, window):
        if self.h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["NVML unavailable: " + getattr(self, "err", "")]}
        self._stop.set()
        self.t.join(timeout=2)
        t0, t1 = self.windows.get(window, (0.0, float("inf")))
        sel = [s for s in self.samples if t0 <= s[0] <= t1] or self.samples
        bits = 0
        for s in sel:
            bits |= s[3]
        allb = 0
        for s in self.samples:
            allb |= s[3]
        return {"sm_mhz": float(np.median([s[1] for s in sel])), "sm_max_mhz": self.max_sm, "samples": len(sel),
                "window": window, "power_w_max": max(s[2] for s in sel),
                "reasons": sorted(k for k, b in self.REASONS.items() if bits & b),
                "whole_run": {"samples": len(self.samples), "sm_mhz": float(np.median([s[1] for s in self.samples])),
                              "power_w_max": max(s[2] for s in self.samples),
                              "reasons": sorted(k for k, b in self.REASONS.items() if allb & b)}}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d["hbm_gbs"], d.get("bf16_tflops_sustained", d.get("bf16_tflops")), "measured"
    return 6650.0, 1400.0, "fallback"


# ------------------------------------------------------------------------------------------ oracle legs

class OracleSample:
    """The CPU oracle, as it stands, on this machine's host cores. It runs `n_layers` decoder layers of the
    workload at full width plus the lm_head; with n_layers = the model's depth that is one whole pass.
    One synthetic layer's weights serve every layer (the arithmetic, and so the time, is the same;
    generating 13-65 GB on the host would take longer than the pass)."""

    def __init__(self, cfg, P, parent, tokens):
        from oracle import oracle as orc
        self.orc, self.cfg, self.P, self.parent, self.tokens = orc, cfg, P, parent, tokens
        self.glob = gen.gen_globals(cfg)
        self.layer = gen.gen_layer(cfg, 0)
        self.pk, self.pv = gen.gen_prefix_kv(cfg, 0, P)

    def run(self, n_layers):
        small = gen.shrink(self.cfg, n_layers)
        lt = []
        t0 = time.perf_counter()
        self.orc.verify_tree(small, self.glob, lambda l: self.layer, lambda l: (self.pk, self.pv), self.P,
                             self.tokens, self.parent, keep_kv=False, layer_times=lt)
        wall = time.perf_counter() - t0
        full = n_layers == self.cfg.n_layers
        if full:
            sec = wall
            desc = (f"one whole pass of the workload by the oracle: all {n_layers} layers at full width + lm_head "
                    f"(N={len(self.tokens)}, P={self.P}), wall time including its fp32 widening of the weights; "
                    "one synthetic layer's weights reused for every layer")
        else:
            sec = float(np.mean(lt[:-1])) * self.cfg.n_layers + lt[-1]
            desc = (f"{n_layers} full-width decoder layer(s) + lm_head of the workload run by the oracle "
                    f"(N={len(self.tokens)}, P={self.P}); per-layer time x {self.cfg.n_layers} layers + head")
        return sec, desc, self.orc.n_threads(), not full


def run_reference(args, w, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    parent = gen.gen_tree(w)
    tokens = gen.gen_tokens(cfg, w.n_nodes)
    smp = OracleSample(cfg, w.prefix_len, parent, tokens)
    layers = cfg.n_layers if args.oracle_layers <= 0 else min(args.oracle_layers, cfg.n_layers)
    times = []
    desc, cores, extrap = "", 0, False
    for i in range(args.warmup + args.steps):
        t, desc, cores, extrap = smp.run(layers)
        if i >= args.warmup:
            times.append(t)
    sec = float(np.median(times))
    val = 1.0 / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "ms_per_step_min": min(times) * 1e3, "ms_per_step_max": max(times) * 1e3,
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "extrapolated": extrap,
        "config": {"workload": workload_name(w, cfg)},
        "tree_tokens_per_sec": val * w.n_nodes,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "extrapolated": extrap},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_name(w, cfg):
    return (f"{w.name}: LLaMA-{cfg.name}-shaped {cfg.dtype} decoder ({cfg.n_layers} layers, d {cfg.d_model}, "
            f"{cfg.n_heads}x{cfg.head_dim} heads, FFN {cfg.d_ffn}, vocab {cfg.vocab}), prefix {w.prefix_len}, "
            f"random draft tree of {w.n_nodes} nodes ({w.branching}, <= {w.max_levels} levels)")


# ------------------------------------------------------------------------------------------ GPU arm

def build_verifier(cfg, w, device, flags=0):
    from paper_2309_04255_b200 import binding as B
    v = B.Verifier(cfg, w.prefix_len + 128 + 8, device=device, flags=flags)
    v.pack_globals({k: gen.gen_tensor_device(cfg, k, -1, device) for k in ("tok_embed", "final_norm", "lm_head")})
    for l in range(cfg.n_layers):
        v.pack_layer(l, {k: gen.gen_tensor_device(cfg, k, l, device) for k in gen.LAYER_TENSORS})
    # synthetic prefix cache ~ N(0,1)
    kvv = v.kv_view()
    g = torch.Generator(device=device)
    g.manual_seed(gen.MASTER_SEED)
    for l in range(cfg.n_layers):
        kvv[l, :, :, : w.prefix_len] = torch.randn((2, cfg.n_heads, w.prefix_len, cfg.head_dim), generator=g,
                                                   device=device, dtype=torch.float32).to(kvv.dtype)
    torch.cuda.synchronize()
    return v


def time_steps(step, steps, barrier):
    """K steps with an event between consecutive steps and no host synchronisation inside: returns the
    per-step milliseconds and the host times of the region's start and end."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    barrier()
    t0 = time.perf_counter()
    ev[0].record()
    for i in range(steps):
        step()
        ev[i + 1].record()
    barrier()
    t1 = time.perf_counter()
    return [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)], ev[0].elapsed_time(ev[steps]), (t0, t1)


def analyze_trace(t, n_layers, passes):
    """t: [launches][256][16] %globaltimer stamps (ns) of `passes` undisturbed passes; per pass the traced
    launches are QKV, then per layer attention, O, gate/up, down, next QKV (lm_head at the end). A launch
    is charged the time from the latest exit seen so far (its predecessor's end) to its own last exit;
    the first launch of a pass from its first entry. The intervals of a pass are disjoint, so their sum is
    at most the pass."""
    per_pass = 1 + 5 * n_layers
    names = ["qkv"] + ["attention", "o", "gate_up", "down", "qkv"] * n_layers
    names[-1] = "lm_head"
    tot = {}
    cnt = {}
    span = 0.0
    for p in range(passes):
        prev = None
        first = None
        for j in range(per_pass):
            sl = t[p * per_pass + j]
            ent = sl[:, 0]
            ext = sl[:, 12]
            ok = ent > 0
            if not ok.any():
                raise RuntimeError(f"launch {j} of pass {p} left no trace")
            e0 = float(ent[ok].min())
            e1 = float(ext[ext > 0].max())
            if prev is None:
                prev, first = e0, e0
            dur = max(0.0, e1 - prev)
            prev = max(prev, e1)
            tot[names[j]] = tot.get(names[j], 0.0) + dur
            cnt[names[j]] = cnt.get(names[j], 0) + 1
        span += prev - first
    out = {k: {"ms_per_step": tot[k] / passes / 1e6, "launches_per_step": cnt[k] // passes,
               "avg_launch_us": tot[k] / cnt[k] / 1e3} for k in tot}
    return out, span / passes / 1e6


def bench_workload(B, v, cfg, w, args, device, barrier, clocks=None, tag="main"):
    """Times one workload on an already built verifier: per-step events, traced passes, isolated launches."""
    P, n = w.prefix_len, w.n_nodes
    rank = int(os.environ.get("RANK", "0"))
    parent_np = gen.gen_tree(w, seed=rank)
    tokens_np = gen.gen_tokens(cfg, n, seed=rank)
    tokens = torch.as_tensor(tokens_np, device=device)
    parent = torch.as_tensor(parent_np, device=device)
    out = v.new_outputs(n, want_logits=True)

    def step():
        v.verify_tree(P, tokens, parent, out=out)

    torch.cuda.synchronize()
    settled_s = clocks.settle() if clocks is not None else 0.0
    for _ in range(args.warmup):
        step()
    barrier()
    sc = out["scalars"].cpu().numpy()
    if int(sc[B.S_STATUS]) != 0:
        raise SystemExit(f"verification pass reported device status {int(sc[B.S_STATUS])}")
    accepted_random = int(sc[B.S_ACCEPTED_LEN])

    # ---- region A: K passes, inputs resident in HBM, an event between consecutive passes
    l0 = v.launch_count()
    per_step, total_ms, win = time_steps(step, args.steps, barrier)
    launches = v.launch_count() - l0
    if clocks is not None:
        clocks.mark(tag, *win)

    res = {"per_step_ms": per_step, "total_ms": total_ms, "launches": int(launches), "accepted_len_random": accepted_random,
           "tokens_np": tokens_np, "parent_np": parent_np, "settled_s": settled_s}

    # ---- region T: the same passes with the kernels' own time stamps (no events between launches)
    if cfg.dtype == "bf16":
        passes = min(args.steps, 8)
        per_pass = 1 + 5 * cfg.n_layers
        buf = torch.zeros((per_pass * passes, 256, 16), dtype=torch.int64, device=device)
        v.set_gemm_trace(buf)
        tr_steps, _, _ = time_steps(step, passes, barrier)
        v.set_gemm_trace(None)
        kinds, span_ms = analyze_trace(buf.cpu().numpy().astype(np.float64), cfg.n_layers, passes)
        del buf
        res["trace"] = {"kinds": kinds, "span_ms_per_step": span_ms, "ms_per_step_traced": float(np.median(tr_steps)), "passes": passes}

    # ---- region B: every GEMM / attention launch bracketed by events (the kernels in isolation)
    v.set_kernel_timing(True)
    iso_steps, _, _ = time_steps(step, min(args.steps, 8), barrier)
    gemm_ms, gemm_cnt = v.get_kernel_timing(0)
    attn_ms, attn_cnt = v.get_kernel_timing(1)
    v.set_kernel_timing(False)
    res["isolated"] = {"gemm_ms": gemm_ms, "gemm_cnt": gemm_cnt, "attn_ms": attn_ms, "attn_cnt": attn_cnt,
                       "steps": len(iso_steps), "ms_per_step": float(np.median(iso_steps))}

    # ---- the planted variant (draft tokens the target really produces along some branches): accepted length
    tok = tokens_np
    o2 = out
    for it in range(6):
        tok = gen.plant_tokens(parent_np, tok, o2["argmax"].cpu().numpy(), seed=it, prob=0.7)
        o2 = v.verify_tree(P, torch.as_tensor(tok, device=device), parent)
    torch.cuda.synchronize()
    res["accepted_len_planted"] = int(o2["scalars"][B.S_ACCEPTED_LEN].item())
    return res


def summarize(cfg, w, res, world, peaks, ms=None, int4=False):
    """ms: the median step time to report (the slowest replica's when there are several)."""
    hbm_peak, tf_peak, peak_kind = peaks
    P, n = w.prefix_len, w.n_nodes
    ab = algorithmic_bytes(cfg, P, n, int4)
    fl = flops(cfg, P, n)
    ms = float(np.median(res["per_step_ms"])) if ms is None else ms
    s = {"ms_per_step": ms, "ms_per_step_min": float(min(res["per_step_ms"])), "ms_per_step_max": float(max(res["per_step_ms"])),
         "ms_per_step_mean": res["total_ms"] / len(res["per_step_ms"]),
         "passes_per_s": world / (ms * 1e-3), "tree_tokens_per_sec": world * n / (ms * 1e-3),
         "pass_hbm_gbs": ab["total"] / (ms * 1e-3) / 1e9,
         "pass_roofline": {"algorithmic_bytes": ab["total"], "flops": fl,
                           "frac_of_measured_hbm": ab["total"] / (ms * 1e-3) / 1e9 / hbm_peak,
                           "frac_of_8TBs": ab["total"] / (ms * 1e-3) / 8e12,
                           "tensor_frac": fl / (ms * 1e-3) / 1e12 / tf_peak, "peaks": peak_kind},
         "accepted_len": {"random_tokens": res["accepted_len_random"], "planted_tokens": res["accepted_len_planted"]}}
    return s


def roofline_block(cfg, w, res, peaks):
    hbm_peak, _, peak_kind = peaks
    n = w.n_nodes
    gb, gcount = gemm_algorithmic_bytes(cfg, n)
    iso = res["isolated"]
    iso_avg_ms = iso["gemm_ms"] / max(iso["gemm_cnt"], 1)
    iso_bytes = gb * iso["steps"] / max(iso["gemm_cnt"], 1)
    iso_gbs = iso_bytes / (iso_avg_ms * 1e-3) / 1e9
    ratio = NCU_GEMM_CAPTURE["dram_bytes"] / NCU_GEMM_CAPTURE["algorithmic_bytes"]
    block = {"kernel": "gemm_stream_kernel (+ gemm_finish_kernel)", "bound": "hbm", "peak": hbm_peak, "unit": "GB/s", "of": peak_kind,
             "algorithmic_bytes_per_launch": gb / gcount, "traffic": ratio * gb / gcount,
             "traffic_source": f"ncu capture {NCU_GEMM_CAPTURE['summary']}: DRAM bytes / algorithmic bytes = {ratio:.3f}, scaled by bytes",
             "isolated": {"achieved": iso_gbs, "frac": iso_gbs / hbm_peak, "avg_launch_ms": iso_avg_ms,
                          "launches_timed": iso["gemm_cnt"], "gemm_ms_per_step": iso["gemm_ms"] / iso["steps"],
                          "attention_ms_per_step": iso["attn_ms"] / iso["steps"], "ms_per_step_with_kernel_events": iso["ms_per_step"],
                          "how": "CUDA events around every launch: no overlap between consecutive kernels"}}
    tr = res.get("trace")
    if tr:
        k = tr["kinds"]
        gemm_ms = sum(v["ms_per_step"] for name, v in k.items() if name != "attention")
        attn_ms = k.get("attention", {"ms_per_step": 0.0})["ms_per_step"]
        avg_ms = gemm_ms / gcount
        ach = gb / (gemm_ms * 1e-3) / 1e9
        block.update({"achieved": ach, "frac": ach / hbm_peak, "avg_launch_ms": avg_ms, "launches_per_step": gcount,
                      "gemm_ms_per_step": gemm_ms, "attention_ms_per_step": attn_ms,
                      "kernels_ms_per_step": gemm_ms + attn_ms, "ms_per_step_traced": tr["ms_per_step_traced"],
                      "per_gemm": {name: {"ms_per_step": v["ms_per_step"], "avg_launch_us": v["avg_launch_us"]} for name, v in k.items()},
                      "how": "inside undisturbed passes: %globaltimer stamps per launch; a launch is charged the time from "
                             "its predecessor's last exit to its own last exit, so kernels_ms_per_step <= ms_per_step_traced"})
    else:
        block.update({"achieved": iso_gbs, "frac": iso_gbs / hbm_peak, "avg_launch_ms": iso_avg_ms})
    return block


def attention_digest(B, device, peaks, reps=30, warmup=5):
    """Config 4 in short: 32 heads x 128, prefix 256..8192 x trees of 8..128 nodes (one random topology
    each), K/V buffers rotated over more than twice the L2 so that every launch reads HBM."""
    from paper_2309_04255_b200 import kernel_bench as KB
    H, hd = 32, 128
    cfg = gen.ModelConfig("attn", 0, H * hd, H, hd, 256, 512, "bf16")
    v = B.Verifier(cfg, 16, device=device)
    cells = []
    for P in (256, 1024, 4096, 8192):
        for n in (8, 32, 64, 128):
            parent = gen.tree_random(n, 16, "uniform4", 0)
            c = KB.attention_cell(v, P, n, parent, reps, warmup, l2_resident=False)
            cells.append({"prefix": P, "nodes": n, "us": round(c["us_attention_kernel"], 2), "gbs": round(c["hbm_gbs"], 1),
                          "frac": round(c["hbm_gbs"] / peaks[0], 4)})
    v.close()
    return {"workload": "C4: tree-masked attention alone, bf16, 32 heads x 128, K/V/Q ~ N(0,1), random trees (branching uniform 1-4)",
            "timing": "CUDA events around each attention launch, K/V rotated over > 2 x L2", "peak_gbs": peaks[0], "cells": cells}


def run_gpu(args, w, cfg):
    from paper_2309_04255_b200 import binding as B
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torchrun for --gpus > 1")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verification pass has no CPU path")
    device = torch.device(f"cuda:{local}")
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    peaks = measured_peaks()
    clocks = ClockSampler(local)
    v = build_verifier(cfg, w, device)
    P, n = w.prefix_len, w.n_nodes
    res = bench_workload(B, v, cfg, w, args, device, barrier, clocks, "timed_region")
    tokens_np, parent_np = res["tokens_np"], res["parent_np"]

    # ---- end to end through the host-buffer entry point (pinned host memory both ways, logits included)
    th = torch.as_tensor(tokens_np).pin_memory()
    ph = torch.as_tensor(parent_np).pin_memory()

    def host_buffers(with_logits):
        return {"logits": torch.empty((n, cfg.vocab), dtype=torch.float32).pin_memory() if with_logits else None,
                "argmax": torch.empty(n, dtype=torch.int32).pin_memory(),
                "accepted_path": torch.empty(128, dtype=torch.int32).pin_memory(),
                "scalars": torch.empty(8, dtype=torch.int32).pin_memory()}

    e2e = {}
    for with_logits in (True, False):
        host = host_buffers(with_logits)
        for _ in range(min(3, args.warmup)):
            v.verify_tree_host(P, th, ph, host)
        barrier()
        ts = []
        for _ in range(args.steps):
            t0 = time.perf_counter()
            v.verify_tree_host(P, th, ph, host)     # synchronises the stream itself
            ts.append(time.perf_counter() - t0)
        e2e[with_logits] = float(np.median(ts)) * 1e3
    clk = clocks.stop("timed_region")
    clk["settled_s"] = round(res["settled_s"], 2)

    ms_med = float(np.median(res["per_step_ms"]))
    times = torch.tensor([ms_med, e2e[True], e2e[False]], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms_med, e2e_ms, e2e_nl_ms = float(times[0]), float(times[1]), float(times[2])

    if rank == 0:
        s = summarize(cfg, w, res, world, peaks, ms=ms_med)
        line = {
            "metric": METRIC, "value": s["passes_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": s["ms_per_step"], "ms_per_step_min": s["ms_per_step_min"], "ms_per_step_max": s["ms_per_step_max"],
            "ms_per_step_mean": s["ms_per_step_mean"], "value_is": "median over the steps",
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": workload_name(w, cfg), "l2": "inputs larger than L2 (weights stream once per pass)",
                       "replicas": world},
            "tree_tokens_per_sec": s["tree_tokens_per_sec"], "pass_hbm_gbs": s["pass_hbm_gbs"],
            "pass_roofline": s["pass_roofline"], "accepted_len": s["accepted_len"],
            "roofline": roofline_block(cfg, w, res, peaks),
            "e2e": {"value": world / (e2e_ms * 1e-3), "unit": UNIT, "logits": True,
                    "h2d_bytes_per_step": 2 * n * 4, "d2h_bytes_per_step": (n + n + 8) * 4 + n * cfg.vocab * 4,
                    "without_logits": {"value": world / (e2e_nl_ms * 1e-3), "d2h_bytes_per_step": (n + n + 8) * 4}},
            "gpu_launches": res["launches"],
            "clocks": clk,
        }
        v.close()
        del v
        torch.cuda.empty_cache()
        if world == 1 and args.extras and w.name == "C2":
            extra = {}
            w3 = gen.WORKLOADS["C3"]
            c3 = gen.MODELS[w3.model]
            v3 = build_verifier(c3, w3, device)
            clocks3 = ClockSampler(local)
            r3 = bench_workload(B, v3, c3, w3, args, device, barrier, clocks3, "timed_region")
            clk3 = clocks3.stop("timed_region")
            s3 = summarize(c3, w3, r3, 1, peaks)
            rb3 = roofline_block(c3, w3, r3, peaks)
            extra["C3"] = {"workload": workload_name(w3, c3), "ms_per_step": s3["ms_per_step"], "ms_per_step_min": s3["ms_per_step_min"],
                           "ms_per_step_max": s3["ms_per_step_max"], "passes_per_s": s3["passes_per_s"],
                           "tree_tokens_per_sec": s3["tree_tokens_per_sec"],
                           "frac_of_measured_hbm": s3["pass_roofline"]["frac_of_measured_hbm"],
                           "frac_of_8TBs": s3["pass_roofline"]["frac_of_8TBs"], "accepted_len": s3["accepted_len"],
                           "gemm_frac_in_pass": rb3.get("frac"), "gemm_ms_per_step": rb3.get("gemm_ms_per_step"),
                           "attention_ms_per_step": rb3.get("attention_ms_per_step"), "steps": args.steps,
                           "clocks": {"sm_mhz": clk3.get("sm_mhz"), "reasons": clk3.get("reasons"), "power_w_max": clk3.get("power_w_max"),
                                      "settled_s": round(r3["settled_s"], 2)}}
            v3.close()
            del v3
            torch.cuda.empty_cache()
            # the benchmarked workload with INT4 weights (Sec. 4.1 of the paper: the target runs INT4 on its devices)
            v4 = build_verifier(cfg, w, device, flags=B.FLAG_INT4_WEIGHTS)
            clocks4 = ClockSampler(local)
            r4 = bench_workload(B, v4, cfg, w, args, device, barrier, clocks4, "timed_region")
            clocks4.stop("timed_region")
            s4 = summarize(cfg, w, r4, 1, peaks, int4=True)
            extra["C2_int4_weights"] = {"workload": workload_name(w, cfg) + "; layer matrices as INT4 codes with power-of-two group scales (groups of 64)",
                                        "ms_per_step": s4["ms_per_step"], "ms_per_step_min": s4["ms_per_step_min"],
                                        "ms_per_step_max": s4["ms_per_step_max"], "passes_per_s": s4["passes_per_s"],
                                        "algorithmic_bytes": s4["pass_roofline"]["algorithmic_bytes"],
                                        "frac_of_measured_hbm": s4["pass_roofline"]["frac_of_measured_hbm"],
                                        "speedup_over_bf16": s["ms_per_step"] / s4["ms_per_step"], "steps": args.steps}
            v4.close()
            del v4
            torch.cuda.empty_cache()
            extra["C4"] = attention_digest(B, device, peaks)
            line["workloads"] = extra
        if world == 1 and not args.no_cpu_baseline:
            smp = OracleSample(cfg, P, parent_np, tokens_np)
            layers = cfg.n_layers if args.oracle_layers <= 0 else min(args.oracle_layers, cfg.n_layers)
            sec, desc, cores, extrap = smp.run(layers)
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                                    "extrapolated": extrap}
        print(json.dumps(line), flush=True)
    else:
        v.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="C2", choices=sorted(gen.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", dest="extras", action="store_false", help="skip the C3 and C4 figures")
    ap.add_argument("--oracle-layers", type=int, default=None,
                    help="decoder layers the oracle runs per step (0 = the whole depth); default: the whole depth for "
                         "C1/C2, 8 layers (extrapolated, and marked so) for the deeper workloads")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = gen.WORKLOADS[args.workload]
    cfg = gen.MODELS[w.model]
    if args.oracle_layers is None:
        args.oracle_layers = 0 if args.workload in ("C1", "C2") else 8
    if args.impl == "reference":
        run_reference(args, w, cfg)
    else:
        run_gpu(args, w, cfg)


if __name__ == "__main__":
    main()
