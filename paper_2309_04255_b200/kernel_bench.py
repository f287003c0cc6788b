"""Single-kernel benchmarks through the C ABI (CUDA events, buffers rotated so that every launch
reads its operands from HBM, not from L2).

    python -m paper_2309_04255_b200.kernel_bench attention            # prefix x tree-size sweep (config 4)
    python -m paper_2309_04255_b200.kernel_bench gemm [--n 32] [--model 7b] [--only qkv,o]
    python -m paper_2309_04255_b200.kernel_bench avnav [--model 7b] [--prefix 512] [--nodes 2,4,...]
    python -m paper_2309_04255_b200.kernel_bench extend [--model 7b] [--prefix 512] [--nodes 32] [--steps 1,2,4,8]
    python -m paper_2309_04255_b200.kernel_bench timeline [--workload C2] [--layers 4] [--int4]   # per-kernel time stamps of one pass
    python -m paper_2309_04255_b200.kernel_bench probes                                            # bulk-copy and mma.sync rates of the machine

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


def attention_cell(v, P, n, parent, reps, warmup, l2_resident=True):
    """One (prefix, tree size) case of the attention-only sweep on verifier `v` (32 heads x 128)."""
    H, hd = v.cfg.n_heads, v.cfg.head_dim
    dev = v.device
    kv_bytes = 2 * H * (P + n) * hd * 2
    io_bytes = kv_bytes + 2 * n * H * hd * 2
    nbuf = max(2, int(2 * L2_BYTES // kv_bytes) + 1)      # rotate over > 2 x L2 of K/V
    g = torch.Generator(device=dev)
    g.manual_seed(gen.MASTER_SEED + P + n)
    ks = [torch.randn((H, P + n, hd), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(nbuf)]
    vs = [torch.randn((H, P + n, hd), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(nbuf)]
    q = torch.randn((n, H, hd), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    par = torch.as_tensor(parent, device=dev)
    us = time_launches(lambda i: v.tree_attention(q, ks[i], vs[i], P, par), nbuf, reps, warmup)
    us_l2 = time_launches(lambda i: v.tree_attention(q, ks[0], vs[0], P, par), 1, reps, warmup) if l2_resident else None
    assert v.last_status() == 0
    # each call is tree-prep + attention; the attention kernel's share is timed by its own events
    v.set_kernel_timing(True)
    for i in range(reps):
        v.tree_attention(q, ks[i % nbuf], vs[i % nbuf], P, par)
    ms, cnt = v.get_kernel_timing(1)
    v.set_kernel_timing(False)
    k_us = ms * 1e3 / max(cnt, 1)
    return {"algorithmic_bytes": io_bytes, "us_per_call_hbm": us, "us_per_call_l2_resident": us_l2,
            "us_attention_kernel": k_us, "hbm_gbs": io_bytes / k_us / 1e3,
            "flops": 4 * n * (P + n) * H * hd, "tflops": 4 * n * (P + n) * H * hd / k_us / 1e6}


def bench_attention(args):
    H, hd = 32, 128
    cfg = gen.ModelConfig("attn", 0, H * hd, H, hd, 256, 512, "bf16")
    v = B.Verifier(cfg, 16)
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
                c = attention_cell(v, P, n, parent, args.reps, args.warmup)
                print(json.dumps({"kernel": "tree_attention", "prefix": P, "nodes": n, "topology": topo, "heads": H, "head_dim": hd,
                                  **c, "peak_gbs": peak, "peak": kind, "frac": c["hbm_gbs"] / peak}), flush=True)


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


def bench_avnav(args):
    """Autoregressive against non-autoregressive verification (Sec. 3.2, the comparison of Fig. 6):
    N tokens verified by N passes of one token each, the prefix growing by one per pass, against one
    pass over a chain of N nodes and one pass over a bushy tree of N nodes. The one-token pass is
    also the plain decoding step of the target model."""
    cfg = gen.MODELS[args.model]
    dev = torch.device("cuda:0")
    P = args.prefix
    sizes = [int(x) for x in args.nodes.split(",")]
    v = B.Verifier(cfg, P + 2 * max(sizes) + 8, device=dev)
    v.pack_globals({k: gen.gen_tensor_device(cfg, k, -1, dev) for k in ("tok_embed", "final_norm", "lm_head")})
    for l in range(cfg.n_layers):
        v.pack_layer(l, {k: gen.gen_tensor_device(cfg, k, l, dev) for k in gen.LAYER_TENSORS})
    kvv = v.kv_view()
    g = torch.Generator(device=dev)
    g.manual_seed(gen.MASTER_SEED)
    for l in range(cfg.n_layers):
        kvv[l, :, :, :P] = torch.randn((2, cfg.n_heads, P, cfg.head_dim), generator=g, device=dev, dtype=torch.float32).to(kvv.dtype)
    peak, kind = _peak()
    wbytes = cfg.weight_bytes()
    root = torch.as_tensor(np.array([-1], np.int32), device=dev)

    def timed(fn, reps):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    for n in sizes:
        tokens = torch.as_tensor(gen.gen_tokens(cfg, n, seed=n), device=dev)
        chain = torch.as_tensor(gen.tree_chain(n), device=dev)
        bushy = torch.as_tensor(gen.tree_random(n, 16, "uniform4", n), device=dev)
        outs1 = [v.new_outputs(1, want_logits=True) for _ in range(n)]
        outn = v.new_outputs(n, want_logits=True)

        def av():
            for i in range(n):
                v.verify_tree(P + i, tokens[i:i + 1], root, out=outs1[i])

        av_ms = timed(av, args.reps)
        step_logits = torch.cat([o["logits"] for o in outs1]).float()
        nav_chain_ms = timed(lambda: v.verify_tree(P, tokens, chain, out=outn), args.reps)
        # the same tokens in one pass must give the same logits as the N one-token passes
        diff = (outn["logits"].float() - step_logits).abs().max().item() / step_logits.abs().max().item()
        nav_tree_ms = timed(lambda: v.verify_tree(P, tokens, bushy, out=outn), args.reps)
        assert v.last_status() == 0
        print(json.dumps({
            "bench": "av_vs_nav", "model": cfg.name, "prefix": P, "nodes": n,
            "av_ms": av_ms, "nav_chain_ms": nav_chain_ms, "nav_tree_ms": nav_tree_ms,
            "speedup_chain": av_ms / nav_chain_ms, "speedup_tree": av_ms / nav_tree_ms,
            "decode_step_ms": av_ms / n, "decode_step_gbs": wbytes / (av_ms / n) / 1e6,
            "decode_step_frac": wbytes / (av_ms / n) / 1e6 / peak, "peak": kind,
            "chain_vs_steps_max_rel_diff": diff}), flush=True)


def build_model(cfg, dev, max_seq, P):
    v = B.Verifier(cfg, max_seq, device=dev)
    v.pack_globals({k: gen.gen_tensor_device(cfg, k, -1, dev) for k in ("tok_embed", "final_norm", "lm_head")})
    for l in range(cfg.n_layers):
        v.pack_layer(l, {k: gen.gen_tensor_device(cfg, k, l, dev) for k in gen.LAYER_TENSORS})
    kvv = v.kv_view()
    g = torch.Generator(device=dev)
    g.manual_seed(gen.MASTER_SEED)
    for l in range(cfg.n_layers):
        kvv[l, :, :, :P] = torch.randn((2, cfg.n_heads, P, cfg.head_dim), generator=g, device=dev, dtype=torch.float32).to(kvv.dtype)
    return v


def bench_extend(args):
    """Tree extension (the generating side's tree decoder): a tree of --nodes nodes grown m nodes at
    a time; every call streams all weights once, like a decoding step."""
    cfg = gen.MODELS[args.model]
    dev = torch.device("cuda:0")
    P, n = args.prefix, args.nodes
    v = build_model(cfg, dev, P + n + 8, P)
    peak, kind = _peak()
    wbytes = cfg.weight_bytes()
    tokens = torch.as_tensor(gen.gen_tokens(cfg, n), device=dev)
    parent = torch.as_tensor(gen.tree_random(n, 16, "uniform4", 1), device=dev)
    for m in [int(x) for x in args.steps.split(",")]:
        cuts = list(range(m, n, m)) + [n]

        def grow():
            old = 0
            for c in cuts:
                v.extend_tree(P, tokens[:c], parent[:c], old, top_k=4, want_logits=False)
                old = c

        grow()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.reps):
            grow()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.reps / len(cuts)
        print(json.dumps({"bench": "extend_tree", "model": cfg.name, "prefix": P, "tree_nodes": n, "new_nodes_per_call": m,
                          "calls": len(cuts), "ms_per_call": ms, "weight_gbs": wbytes / ms / 1e6,
                          "frac": wbytes / ms / 1e6 / peak, "peak": kind}), flush=True)


def bench_timeline(args):
    """One undisturbed pass of a workload (a few layers of its model) with the kernels' own %globaltimer
    stamps (llmcad_set_gemm_trace): where every GEMM's streaming kernel (S) and finishing kernel (F) and
    every attention kernel starts, sees its dependency, ends; a launch is charged the time from its
    predecessor's end to its own. Microseconds since the first stamp, median over the CTAs unless a
    range min..max is given."""
    dev = torch.device("cuda:0")
    w = gen.WORKLOADS[args.workload]
    L = args.layers
    cfg = gen.shrink(gen.MODELS[w.model], L)
    P, n = w.prefix_len, w.n_nodes
    v = B.Verifier(cfg, P + 136, device=dev, flags=B.FLAG_INT4_WEIGHTS if args.int4 else 0)
    v.pack_globals({k: gen.gen_tensor_device(cfg, k, -1, dev) for k in ("tok_embed", "final_norm", "lm_head")})
    for l in range(L):
        v.pack_layer(l, {k: gen.gen_tensor_device(cfg, k, l, dev) for k in gen.LAYER_TENSORS})
    kvv = v.kv_view()
    kvv[:, :, :, :P] = torch.randn((L, 2, cfg.n_heads, P, cfg.head_dim), device=dev).to(kvv.dtype)
    tokens = torch.as_tensor(gen.gen_tokens(cfg, n), device=dev)
    parent = torch.as_tensor(gen.gen_tree(w), device=dev)
    out = v.new_outputs(n)
    for _ in range(3):
        v.verify_tree(P, tokens, parent, out=out)
    torch.cuda.synchronize()
    cap = 1 + 5 * L
    buf = torch.zeros(cap, 256, 16, dtype=torch.int64, device=dev)
    v.set_gemm_trace(buf)
    v.verify_tree(P, tokens, parent, out=out)
    torch.cuda.synchronize()
    v.set_gemm_trace(None)
    t = buf.cpu().numpy().astype(np.float64)
    names = ["qkv"] + ["attention", "o", "gate_up", "down", "qkv"] * L
    names[-1] = "lm_head"
    base = t[0][:, 0][t[0][:, 0] > 0].min()

    def st(T, slot):
        x = T[:, slot]
        x = x[x > 0]
        return ((x.min() - base) / 1e3, (np.median(x) - base) / 1e3, (x.max() - base) / 1e3) if len(x) else (-1.0, -1.0, -1.0)

    prev = 0.0
    for i in range(cap):
        T = t[i]
        end = st(T, 12)[2]
        row = {"launch": i, "kernel": names[i], "charged_us": round(end - prev, 2)}
        prev = end
        if names[i] == "attention":
            keys = {"entry": 0, "dependency": 1, "first_tile": 2, "loop_end": 3, "cta_merged": 4, "cluster_sync": 5, "stored": 6, "exit": 12}
        else:
            keys = {"S_entry": 0, "S_first_copy": 2, "S_dependency": 3, "S_last_copy": 6, "S_last_mma": 7, "S_dumped": 8, "S_exit": 13,
                    "F_entry": 9, "F_dependency": 10, "F_exit": 12}
        for k, slot in keys.items():
            a, m, b = st(T, slot)
            row[k] = f"{m:.2f} ({a:.2f}..{b:.2f})"
        print(json.dumps(row), flush=True)


def bench_probes(args):
    """What the machine gives to the two access patterns of the pass (llmcad_probe_* of the measurement interface):
    cp.async.bulk copies streaming a buffer of 8 GB from HBM once, by copy size and copies in flight per SM; and the
    legacy mma.sync.m16n8k16 bf16 path by warps per SM and independent accumulators per warp."""
    dev = torch.device("cuda:0")
    src = torch.empty(args.gb << 30, dtype=torch.uint8, device=dev)
    src.fill_(1)
    torch.cuda.synchronize()
    for size in (4224, 8448, 16384, 32768):
        for depth in (1, 2, 4, 8, 12):
            if size * depth > 200 * 1024:
                continue
            B.probe_bulk_copy(src, size, depth)          # warm-up
            gbs, lat = B.probe_bulk_copy(src, size, depth)
            print(json.dumps({"probe": "bulk_copy", "copy_bytes": size, "in_flight": depth, "gbs": round(gbs, 1),
                              "latency_us": round(lat, 2)}), flush=True)
    for warps, acc in ((1, 1), (8, 1), (8, 2), (8, 4), (8, 8), (16, 8), (4, 8)):
        rate, cyc = B.probe_mma_sync(warps, acc)
        print(json.dumps({"probe": "mma_sync_m16n8k16_bf16", "warps_per_sm": warps, "accumulators_per_warp": acc,
                          "fma_per_clk_sm": round(rate, 1), "cycles_per_mma_per_warp": round(cyc, 1)}), flush=True)


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
    n = sub.add_parser("avnav")
    n.add_argument("--model", default="7b")
    n.add_argument("--prefix", type=int, default=512)
    n.add_argument("--nodes", default="2,4,8,16,32,64,128")
    n.add_argument("--reps", type=int, default=3)
    x = sub.add_parser("extend")
    x.add_argument("--model", default="7b")
    x.add_argument("--prefix", type=int, default=512)
    x.add_argument("--nodes", type=int, default=32)
    x.add_argument("--steps", default="1,2,4,8,32")
    x.add_argument("--reps", type=int, default=3)
    t = sub.add_parser("timeline")
    t.add_argument("--workload", default="C2")
    t.add_argument("--layers", type=int, default=4)
    t.add_argument("--int4", action="store_true")
    pr = sub.add_parser("probes")
    pr.add_argument("--gb", type=int, default=8)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("kernel_bench needs a CUDA device")
    {"attention": bench_attention, "gemm": bench_gemm, "avnav": bench_avnav, "extend": bench_extend,
     "timeline": bench_timeline, "probes": bench_probes}[args.cmd](args)


if __name__ == "__main__":
    main()
