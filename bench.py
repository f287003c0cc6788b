#!/usr/bin/env python
"""Benchmark of the token-tree verification pass (one step = one whole pass: mask table, decoder
forward over all tree nodes, argmax, verified-path search, cache rollback).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2|C3|C5|C1] [--impl reference]

Prints ONE JSON line. The path does not shard (one GPU per model replica, no collective): with
--gpus N > 1, launched under torchrun, every rank runs an independent replica of the same
workload and the value is the replicas' total.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2309_04255_b200 import inputs as gen  # noqa: E402

METRIC = "tree_verification_passes_per_sec"
UNIT = "passes/s"
# ncu capture of gemm_chain_kernel (profiles/gemm_chain_kernel__7b_qkv_n32.md): DRAM bytes per launch relative to the launch's
# algorithmic bytes; None until a capture exists for the workload.
GEMM_TRAFFIC_RATIO = 1.02


def algorithmic_bytes(cfg, P, n):
    """Bytes one pass must move: every weight matrix once, the prefix K/V once, the tree nodes'
    K/V written and read once, the embedding rows of the n tokens, the fp32 logits."""
    e = cfg.elem_bytes
    weights = cfg.weight_bytes()
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
    """nvidia-smi clock / throttle-reason samples during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [r.split(", ") for r in open(self.f.name).read().strip().splitlines() if r.strip()]
        os.unlink(self.f.name)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[1])); smax.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for nm, val in zip(names, r[5:9]):
                if val.strip().lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d["hbm_gbs"], d.get("bf16_tflops_sustained", d.get("bf16_tflops")), "measured"
    return 6650.0, 1400.0, "fallback"


# ------------------------------------------------------------------------------------------ oracle legs

class OracleSample:
    """The CPU oracle, as it stands, on a bounded sample of the workload: `n_layers` decoder layers
    at full width plus the lm_head, on this machine's host cores; the per-layer time is extrapolated
    to the model's depth (every layer costs the same arithmetic)."""

    def __init__(self, cfg, P, parent, tokens):
        from oracle import oracle as orc
        self.orc, self.cfg, self.P, self.parent, self.tokens = orc, cfg, P, parent, tokens
        self.glob = gen.gen_globals(cfg)
        self.layer = gen.gen_layer(cfg, 0)              # one synthetic layer, reused for every sample layer
        self.pk, self.pv = gen.gen_prefix_kv(cfg, 0, P)

    def run(self, n_layers):
        small = gen.shrink(self.cfg, n_layers)
        lt = []
        self.orc.verify_tree(small, self.glob, lambda l: self.layer, lambda l: (self.pk, self.pv), self.P,
                             self.tokens, self.parent, keep_kv=False, layer_times=lt)
        sec = float(np.mean(lt[:-1])) * self.cfg.n_layers + lt[-1]
        desc = (f"{n_layers} full-width decoder layer(s) + lm_head of the workload run by the oracle "
                f"(N={len(self.tokens)}, P={self.P}); per-layer time x {self.cfg.n_layers} layers + head")
        return sec, desc, self.orc.n_threads()


def run_reference(args, w, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    parent = gen.gen_tree(w)
    tokens = gen.gen_tokens(cfg, w.n_nodes)
    smp = OracleSample(cfg, w.prefix_len, parent, tokens)
    times = []
    desc, cores = "", 0
    for i in range(args.warmup + args.steps):
        t, desc, cores = smp.run(1)
        if i >= args.warmup:
            times.append(t)
    sec = float(np.mean(times))
    val = 1.0 / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(w, cfg)},
        "tree_tokens_per_sec": val * w.n_nodes,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_name(w, cfg):
    return (f"{w.name}: LLaMA-{cfg.name}-shaped {cfg.dtype} decoder ({cfg.n_layers} layers, d {cfg.d_model}, "
            f"{cfg.n_heads}x{cfg.head_dim} heads, FFN {cfg.d_ffn}, vocab {cfg.vocab}), prefix {w.prefix_len}, "
            f"random draft tree of {w.n_nodes} nodes ({w.branching}, <= {w.max_levels} levels)")


# ------------------------------------------------------------------------------------------ GPU arm

def build_verifier(cfg, w, device):
    from paper_2309_04255_b200 import binding as B
    v = B.Verifier(cfg, w.prefix_len + 128 + 8, device=device)
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

    v = build_verifier(cfg, w, device)
    P, n = w.prefix_len, w.n_nodes
    parent_np = gen.gen_tree(w, seed=rank)
    tokens_np = gen.gen_tokens(cfg, n, seed=rank)
    tokens = torch.as_tensor(tokens_np, device=device)
    parent = torch.as_tensor(parent_np, device=device)
    out = v.new_outputs(n, want_logits=True)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def step():
        v.verify_tree(P, tokens, parent, out=out)

    for _ in range(args.warmup):
        step()
    barrier()
    st = int(out["scalars"][B.S_STATUS].item())
    if st != 0:
        raise SystemExit(f"verification pass reported device status {st}")

    # ---- timed region A: K passes, inputs resident in HBM, CUDA events on the launching stream
    clocks = ClockSampler(local)
    l0 = v.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = v.launch_count() - l0

    # ---- timed region B: the same K passes with every GEMM / attention launch bracketed by events
    v.set_kernel_timing(True)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(args.steps):
        step()
    f1.record()
    barrier()
    gemm_ms, gemm_cnt = v.get_kernel_timing(0)
    attn_ms, attn_cnt = v.get_kernel_timing(1)
    v.set_kernel_timing(False)
    ms_events = f0.elapsed_time(f1)

    # ---- end to end through the host-buffer entry point (pinned host memory both ways)
    th = torch.as_tensor(tokens_np).pin_memory()
    ph = torch.as_tensor(parent_np).pin_memory()
    host = {"logits": None, "argmax": torch.empty(n, dtype=torch.int32).pin_memory(),
            "accepted_path": torch.empty(128, dtype=torch.int32).pin_memory(),
            "scalars": torch.empty(8, dtype=torch.int32).pin_memory()}
    for _ in range(min(3, args.warmup)):
        v.verify_tree_host(P, th, ph, host)
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        v.verify_tree_host(P, th, ph, host)     # synchronises the stream itself
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    clk = clocks.stop()

    times = torch.tensor([ms, e2e_s * 1e3], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms, e2e_ms = float(times[0]), float(times[1])

    if rank == 0:
        hbm_peak, tf_peak, peak_kind = measured_peaks()
        ab = algorithmic_bytes(cfg, P, n)
        gb, gcount = gemm_algorithmic_bytes(cfg, n)
        ms_per = ms / args.steps
        value = world * args.steps / (ms * 1e-3)
        gemm_avg_ms = gemm_ms / max(gemm_cnt, 1)
        gb_launch = gb * args.steps / max(gemm_cnt, 1)          # a launch may chain several GEMMs
        gemm_gbs = gb_launch / (gemm_avg_ms * 1e-3) / 1e9
        fl = flops(cfg, P, n)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": workload_name(w, cfg), "l2": "inputs larger than L2 (weights stream once per pass)",
                       "replicas": world},
            "tree_tokens_per_sec": value * n,
            "pass_hbm_gbs": ab["total"] / (ms_per * 1e-3) / 1e9,
            "pass_roofline": {"algorithmic_bytes": ab["total"], "flops": fl,
                              "frac_of_measured_hbm": ab["total"] / (ms_per * 1e-3) / 1e9 / hbm_peak,
                              "frac_of_8TBs": ab["total"] / (ms_per * 1e-3) / 8e12,
                              "tensor_frac": fl / (ms_per * 1e-3) / 1e12 / tf_peak, "peaks": peak_kind},
            "roofline": {"kernel": "gemm_chain_kernel", "bound": "hbm", "achieved": gemm_gbs, "peak": hbm_peak,
                         "unit": "GB/s", "frac": gemm_gbs / hbm_peak,
                         "traffic": (GEMM_TRAFFIC_RATIO * gb_launch) if GEMM_TRAFFIC_RATIO else None,
                         "launches_timed": gemm_cnt, "avg_launch_ms": gemm_avg_ms,
                         "algorithmic_bytes_per_launch": gb_launch, "of": peak_kind,
                         "ms_per_step_with_kernel_events": ms_events / args.steps,
                         "attention_ms_per_step": attn_ms / args.steps, "gemm_ms_per_step": gemm_ms / args.steps},
            "e2e": {"value": world * args.steps / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": 2 * n * 4, "d2h_bytes_per_step": (n + n + 8) * 4},
            "gpu_launches": int(launches),
            "clocks": clk,
        }
        if world == 1 and not args.no_cpu_baseline:
            sec, desc, cores = OracleSample(cfg, P, parent_np, tokens_np).run(args.oracle_layers)
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        print(json.dumps(line), flush=True)
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
    ap.add_argument("--oracle-layers", type=int, default=8)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = gen.WORKLOADS[args.workload]
    cfg = gen.MODELS[w.model]
    if args.impl == "reference":
        run_reference(args, w, cfg)
    else:
        run_gpu(args, w, cfg)


if __name__ == "__main__":
    main()
