"""CPU-side checks: the C-ABI library loads and exports every symbol the header declares, the
binding marshals what the header says, the input generators are deterministic, and the
multi-replica timing reduction used by bench.py works across processes (gloo, world size 2)."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

from paper_2309_04255_b200 import inputs as gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    """Every function declared in include/*.h (the pass itself and the measurement interface)."""
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if f.endswith(".h"):
            src = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, f)).read(), flags=re.S)
            names |= set(re.findall(r"\b(llmcad_[a-z_0-9]+)\s*\(", src))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    from paper_2309_04255_b200 import build as libbuild
    lib = ctypes.CDLL(libbuild.build())
    names = header_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/*.h but not exported"
    lib.llmcad_strerror.restype = ctypes.c_char_p
    assert lib.llmcad_version() >= 100
    assert lib.llmcad_strerror(-3) == b"prefix_len + n exceeds the cache capacity"
    assert lib.llmcad_strerror(1) == b"malformed tree (parent_idx)"


def test_binding_lists_the_same_symbols():
    from paper_2309_04255_b200 import binding as B
    assert sorted(B.EXPORTS) == header_functions()
    # struct layouts agree with the header (field order and count)
    assert [f[0] for f in B.Config._fields_] == ["n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab",
                                                   "max_seq", "max_tree", "rms_eps", "rope_base", "dtype", "flags"]
    assert ctypes.sizeof(B.Config) == 48
    assert ctypes.sizeof(B.LayerWeights) == 9 * 8 and ctypes.sizeof(B.Result) == 4 * 8


def test_size_queries_without_a_gpu():
    """Pure host arithmetic of the ABI: cache and packed-weight sizes, argument validation."""
    from paper_2309_04255_b200 import binding as B
    cfg = gen.MODELS["7b"]
    c = B.make_config(cfg, 1024)
    L = B.lib()
    assert L.llmcad_kv_cache_bytes(ctypes.byref(c)) == 32 * 2 * 32 * 1024 * 128 * 2
    packed = L.llmcad_packed_weight_bytes(ctypes.byref(c))
    assert packed >= cfg.weight_bytes() + cfg.vocab * cfg.d_model * 2          # + embedding
    assert packed < 1.001 * (cfg.weight_bytes() + cfg.vocab * cfg.d_model * 2) + (1 << 20)
    bad = B.make_config(cfg, 1024)
    bad.head_dim = 96
    assert L.llmcad_kv_cache_bytes(ctypes.byref(bad)) == 0
    h = ctypes.c_void_p()
    assert L.llmcad_create(ctypes.byref(bad), ctypes.byref(h)) == B.ERR_UNSUPPORTED
    assert L.llmcad_create(None, ctypes.byref(h)) == B.ERR_INVALID_ARG


def test_no_cpu_fallback():
    """Without a CUDA device the product path refuses to run instead of computing elsewhere."""
    import torch
    from paper_2309_04255_b200 import binding as B
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        B.Verifier(gen.MODELS["tiny"], 64)
    c = B.make_config(gen.MODELS["tiny"], 64)
    h = ctypes.c_void_p()
    assert B.lib().llmcad_create(ctypes.byref(c), ctypes.byref(h)) == B.ERR_CUDA


def test_product_path_does_not_import_the_oracle():
    for root, _, files in os.walk(os.path.join(ROOT, "paper_2309_04255_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(root, f)).read()
                assert "oracle" not in txt.lower() or f == "inputs.py", f
    assert "import oracle" not in open(os.path.join(ROOT, "paper_2309_04255_b200", "inputs.py")).read()


def test_generators_are_deterministic_and_shaped_like_the_workloads():
    cfg = gen.MODELS["tiny"]
    a, b = gen.gen_layer(cfg, 1), gen.gen_layer(cfg, 1)
    assert all((a[k] == b[k]).all() for k in a)
    assert not (gen.gen_layer(cfg, 0)["wq"] == a["wq"]).all()
    assert abs(float(a["w_down"].std()) - 0.02) < 1e-3 and a["w_down"].shape == (256, 688)
    assert (a["attn_norm"] == 1).all()
    for name, w in gen.WORKLOADS.items():
        p = gen.gen_tree(w)
        assert len(p) == w.n_nodes and p[0] == -1 and all(0 <= p[i] < i for i in range(1, len(p)))
        depth = np.zeros(len(p), int)
        for i in range(1, len(p)):
            depth[i] = depth[p[i]] + 1
        assert depth.max() + 1 <= w.max_levels
        assert (p == gen.gen_tree(w)).all()
    assert np.bincount(gen.gen_tree(gen.WORKLOADS["C2"])[1:]).max() <= 4


_WORKER = r'''
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
# each replica reports its own elapsed time; the job's time is the slowest replica's
ms = torch.tensor([10.0 + 5.0 * rank, 3.0], dtype=torch.float64)
dist.barrier()
dist.all_reduce(ms, op=dist.ReduceOp.MAX)
steps, world = 4, dist.get_world_size()
value = world * steps / (ms[0].item() * 1e-3)
if rank == 0:
    print("VALUE", value, ms.tolist())
dist.destroy_process_group()
'''


def test_replica_aggregation_world_size_2(tmp_path):
    """bench.py --gpus N runs independent replicas (no collective on the data path): the reported
    value is the replicas' total steps over the max-over-ranks time. Same reduction, gloo on CPU."""
    script = tmp_path / "w.py"
    script.write_text(_WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29617", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script), ROOT], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    line = [l for l in outs[0][0].splitlines() if l.startswith("VALUE")][0].split(None, 2)
    assert abs(float(line[1]) - 2 * 4 / 15e-3) < 1e-6


def test_bench_reference_arm_runs_on_cpu():
    """`bench.py --impl reference` times the oracle on host cores; tiny workload here."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    import json
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["unit"] == "passes/s"


def test_fallback_scalars_match_the_oracle():
    """llmcad_update_threshold / llmcad_tree_confidence (host arithmetic of Eq. 3) against the oracle
    on a grid of cases, and their argument checks."""
    from oracle import oracle as orc
    from paper_2309_04255_b200 import binding as B
    rng = np.random.default_rng(11)
    for _ in range(200):
        n_all = int(rng.integers(0, 12))
        n_correct = int(rng.integers(0, n_all + 1))
        t_c = float(rng.uniform(1e-3, 1.0))
        alpha = float(rng.uniform(1e-4, 0.5))
        got = B.update_threshold(alpha, n_correct, n_all, t_c)
        ref = orc.alpha_update(alpha, n_correct, n_all, t_c)
        assert abs(got - ref) <= 1e-12 * abs(ref)
    c = rng.uniform(0.01, 1.0, 9)
    assert B.tree_confidence(c) == orc.tree_confidence(c)
    for bad in [(0.0, 1, 2, 0.5), (0.01, 3, 2, 0.5), (0.01, -1, 2, 0.5), (0.01, 1, 2, 0.0), (0.01, 1, 2, 1.5)]:
        with pytest.raises(B.LlmcadError):
            B.update_threshold(*bad)
    with pytest.raises(B.LlmcadError):
        B.tree_confidence([0.5, 0.0])


def test_branch_pacer_matches_the_oracle():
    """llmcad_tree_branches / llmcad_branch_pacer (host arithmetic of Eq. 1-2) against the oracle on
    random trees, and their argument checks."""
    from oracle import oracle as orc
    from paper_2309_04255_b200 import binding as B
    from paper_2309_04255_b200 import inputs as gen
    rng = np.random.default_rng(21)
    for n in (1, 2, 5, 32, 77, 128):
        for shape in ("uniform4", "geometric4", "chain"):
            parent = np.arange(-1, n - 1) if shape == "chain" else gen.tree_random(n, 10, shape, n)
            conf = rng.uniform(0.02, 1.0, n)
            leaf, cum, length = B.tree_branches(parent, conf)
            o_leaf, o_cum, o_len = orc.tree_branches(parent, conf)
            assert leaf == o_leaf.tolist() and length == o_len.tolist()
            np.testing.assert_allclose(cum, o_cum, rtol=1e-12)
            m = float(sum(length)) + float(rng.integers(0, 4))
            f, nxt = B.branch_pacer(cum, length, m)
            o_f, o_nxt = orc.branch_pacer(o_cum, o_len, m)
            np.testing.assert_allclose(f, o_f, rtol=1e-12, atol=1e-12)
            if np.sort(o_f)[-1] - (np.sort(o_f)[-2] if len(o_f) > 1 else -np.inf) > 1e-9:
                assert nxt == o_nxt                       # a unique maximum must be found by both
            else:
                assert abs(f[nxt] - o_f.max()) <= 1e-9
    for bad in [([0, 0], [1.0, 0.5]), ([-1, 1], [1.0, 0.5]), ([-1, 0], [1.0, 0.0]), ([-1, 0], [1.0, 1.5]), ([-1] * 129, [0.5] * 129)]:
        with pytest.raises(B.LlmcadError):
            B.tree_branches(*bad)
    for bad in [([0.5, 0.0], [1, 1], 2), ([0.5, 0.5], [1, -1], 2), ([0.5, 0.5], [1, 1], -1.0)]:
        with pytest.raises(B.LlmcadError):
            B.branch_pacer(*bad)
