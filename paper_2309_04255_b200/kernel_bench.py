"""Single-kernel benchmarks through the C ABI (CUDA events, buffers rotated so that every launch
reads its operands from HBM, not from L2).

    python -m paper_2309_04255_b200.kernel_bench attention            # prefix x tree-size sweep (config 4)
    python -m paper_2309_04255_b200.kernel_bench gemm [--n 32] [--model 7b] [--only qkv,o]

Each line of output is one JSON object. `--reps` launches are timed per case after `--warmup`.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2309_04255_b200 import binding as B  # noqa: E402
from paper_2309_04255_b200 import inputs as gen  # noqa: E402

L2_BYTES = 126e6


def _peak():
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p))["hbm_gbs"], "measured"
    return 6650.0, "fallback"


def time_launches(fn, n_variants, reps, warmup):
    for i in range(warmup):
        fn(i % n_variants)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        fn(i % n_variants)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps      # microseconds per launch


def bench_attention(args):
    H, hd = 32, 128
    cfg = gen.ModelConfig("attn", 0, H * hd, H, hd, 256, 512, "bf16")
    v = B.Verifier(cfg, 16)
    dev = v.device
    peak, kind = _peak()
    prefixes = [int(x) for x in args.prefix.split(",")]
    sizes = [int(x) for x in args.nodes.split(",")]
    for P in prefixes:
        for n in sizes:
            for topo in args.topologies.split(","):
                if topo == "chain":
                    parent = gen.tree_chain(n)
                elif topo == "star":
                    parent = gen.tree_star(n)
                else:
                    parent = gen.tree_random(n, 16, "uniform4", int(topo)) if n > 1 else np.array([-1], np.int32)
                kv_bytes = 2 * H * (P + n) * hd * 2
                io_bytes = kv_bytes + 2 * n * H * hd * 2
                nbuf = max(2, int(2 * L2_BYTES // kv_bytes) + 1)      # rotate over > 2 x L2 of K/V
                g = torch.Generator(device=dev)
                g.manual_seed(gen.MASTER_SEED + P + n)
                ks = [torch.randn((H, P + n, hd), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(nbuf)]
                vs = [torch.randn((H, P + n, hd), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(nbuf)]
                q = torch.randn((n, H, hd), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
                par = torch.as_tensor(parent, device=dev)
                us = time_launches(lambda i: v.tree_attention(q, ks[i], vs[i], P, par), nbuf, args.reps, args.warmup)
                us_l2 = time_launches(lambda i: v.tree_attention(q, ks[0], vs[0], P, par), 1, args.reps, args.warmup)
                assert v.last_status() == 0
                # each call is tree-prep + attention; the attention kernel's share is timed by its own events
                v.set_kernel_timing(True)
                for i in range(args.reps):
                    v.tree_attention(q, ks[i % nbuf], vs[i % nbuf], P, par)
                ms, cnt = v.get_kernel_timing(1)
                v.set_kernel_timing(False)
                k_us = ms * 1e3 / max(cnt, 1)
                print(json.dumps({
                    "kernel": "tree_attention", "prefix": P, "nodes": n, "topology": topo, "heads": H, "head_dim": hd,
                    "algorithmic_bytes": io_bytes, "us_per_call_hbm": us, "us_per_call_l2_resident": us_l2,
                    "us_attention_kernel": k_us, "hbm_gbs": io_bytes / k_us / 1e3, "peak_gbs": peak, "peak": kind,
                    "frac": io_bytes / k_us / 1e3 / peak,
                    "flops": 4 * n * (P + n) * H * hd, "tflops": 4 * n * (P + n) * H * hd / k_us / 1e6}), flush=True)
                del ks, vs


def bench_gemm(args):
    m = gen.MODELS[args.model]
    d, f, V = m.d_model, m.d_ffn, m.vocab
    shapes = {"qkv": (3 * d, d), "o": (d, d), "gate_or_up": (f, d), "down": (d, f), "lm_head": (V, d)}
    only = args.only.split(",") if args.only else list(shapes)
    cfg = gen.ModelConfig("gemm", 0, 256, 2, 128, 256, 512, "bf16")
    v = B.Verifier(cfg, 16)
    dev = v.device
    peak, kind = _peak()
    n = args.n
    for name in only:
        n_out, n_in = shapes[name]
        wbytes = n_out * n_in * 2
        nbuf = max(2, int(2 * L2_BYTES // wbytes) + 1)
        g = torch.Generator(device=dev)
        g.manual_seed(gen.MASTER_SEED + n_out)
        Ws = []
        for _ in range(nbuf):   # the layout the pass streams: pre-swizzled 16 KB tiles
            Ws.append(v.tile_weight((torch.randn((n_out, n_in), generator=g, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)))
        x = torch.randn((n, n_in), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
        us = time_launches(lambda i: v.skinny_gemm_tiled(Ws[i], n_out, x), nbuf, args.reps, args.warmup)
        assert v.last_status() == 0
        v.set_kernel_timing(True)
        for i in range(args.reps):
            v.skinny_gemm_tiled(Ws[i % nbuf], n_out, x)
        ms, cnt = v.get_kernel_timing(0)
        v.set_kernel_timing(False)
        k_us = ms * 1e3 / max(cnt, 1)
        by = wbytes + n * n_in * 2 + n * n_out * 4
        print(json.dumps({"kernel": "skinny_gemm", "name": name, "n_out": n_out, "n_in": n_in, "nodes": n,
                          "algorithmic_bytes": by, "us_per_call": us, "us_gemm_kernel": k_us,
                          "hbm_gbs": by / k_us / 1e3, "peak_gbs": peak, "peak": kind, "frac": by / k_us / 1e3 / peak,
                          "tflops": 2 * n * n_out * n_in / k_us / 1e6}), flush=True)
        del Ws


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    a = sub.add_parser("attention")
    a.add_argument("--prefix", default="256,1024,4096,8192")
    a.add_argument("--nodes", default="8,32,64,128")
    a.add_argument("--topologies", default="0", help="comma list of seeds, or chain / star")
    a.add_argument("--reps", type=int, default=50)
    a.add_argument("--warmup", type=int, default=5)
    g = sub.add_parser("gemm")
    g.add_argument("--n", type=int, default=32)
    g.add_argument("--model", default="7b")
    g.add_argument("--only", default="")
    g.add_argument("--reps", type=int, default=30)
    g.add_argument("--warmup", type=int, default=5)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("kernel_bench needs a CUDA device")
    (bench_attention if args.cmd == "attention" else bench_gemm)(args)


if __name__ == "__main__":
    main()
