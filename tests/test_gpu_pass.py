"""Whole-pass GPU parity against the CPU oracle on seeded inputs, through the C ABI.

Tolerances (from the benchmark spec): indexing bit-exact; fp32 logits max|delta| <= 1e-4 *
max|logit|; bf16 logits max|delta| <= 2e-2 * max|logit| with argmax agreement wherever the top-2
margin exceeds that bound."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2309_04255_b200 import binding as B
from paper_2309_04255_b200 import inputs as gen

from gpu_util import (BF16_TOL, F32_TOL, Twin, argmax_agrees_where_decided, cache_rows,
                      check_acceptance_against_oracle, logits_close)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def oracle_prefill(twin, prefix_tokens, max_seq):
    dec = orc.SequentialDecoder(twin.cfg, twin.glob, [twin.layer(l) for l in range(twin.cfg.n_layers)], max_seq)
    last = None
    for t in prefix_tokens:
        last = dec.step(int(t))
    return dec, last


def compare_cache(twin, dec_or_rows, upto, tol):
    got = cache_rows(twin.v, upto)                       # [L][2][H][upto][hd]
    for l in range(twin.cfg.n_layers):
        k, v = dec_or_rows(l)
        for which, ref in ((0, k), (1, v)):
            scale = np.abs(ref).max()
            assert np.abs(got[l, which] - ref).max() <= tol * scale


# ----------------------------------------------------------------------------- config 1 (fp32)

@pytest.mark.parametrize("scale", [1.0, 6.0])
def test_c1_tiny_fp32_whole_pass(scale):
    """Config 1: 2 layers, d 256, 4x64 heads, FFN 688, vocab 1024, prefix 32 (real prefill on both
    sides), full binary tree of 15 nodes; then a planted variant with a non-trivial verified path."""
    w = gen.WORKLOADS["C1"]
    cfg = gen.MODELS[w.model]
    twin = Twin(cfg, 64, scale=scale)
    prefix = gen.gen_prefix_tokens(cfg, w.prefix_len)
    parent = gen.gen_tree(w)
    tokens = gen.gen_tokens(cfg, w.n_nodes)
    P = w.prefix_len

    dec, last = oracle_prefill(twin, prefix, 64)
    lg = twin.v.prefill(0, torch.as_tensor(prefix, device=DEV), want_logits=True)
    assert twin.v.last_status() == 0
    logits_close(lg.cpu().numpy()[None], last[None], F32_TOL)
    compare_cache(twin, lambda l: dec.cache_heads(l, P), P, 1e-5)

    def both(tok):
        ref = orc.verify_tree(cfg, twin.glob, twin.layer, lambda l: dec.cache_heads(l, P), P, tok, parent)
        out = twin.gpu_pass(P, tok, parent)
        logits_close(out["logits"], ref.logits, F32_TOL)
        return ref, out

    ref, out = both(tokens)
    assert (out["argmax"] == ref.argmax).all()
    acc = check_acceptance_against_oracle(out, tokens, parent)
    assert acc.path.tolist() == ref.acceptance.path.tolist()

    # planted: draft tokens that the target really produces along some branches
    tok = tokens
    for it in range(5):
        tok = gen.plant_tokens(parent, tok, ref.argmax, seed=it, prob=0.9)
        ref = orc.verify_tree(cfg, twin.glob, twin.layer, lambda l: dec.cache_heads(l, P), P, tok, parent)
    ref, out = both(tok)
    assert ref.acceptance.accepted_len >= 2
    assert (out["argmax"] == ref.argmax).all()
    acc = check_acceptance_against_oracle(out, tok, parent)
    assert acc.path.tolist() == ref.acceptance.path.tolist()
    assert out["scalars"][B.S_NEW_PREFIX_LEN] == ref.new_prefix_len
    # rolled-back cache == prefix rows + the verified nodes' rows (oracle K/V, fp32 tolerance)
    def rows(l):
        pk, pv = dec.cache_heads(l, P)
        return (orc.compact(pk, ref.tree_k[l], acc.path, cfg.n_heads, cfg.head_dim),
                orc.compact(pv, ref.tree_v[l], acc.path, cfg.n_heads, cfg.head_dim))
    compare_cache(twin, rows, ref.new_prefix_len, 1e-5)


def test_c1_chain_equals_repeated_single_token_passes():
    """One-shot verification gives what examining the tokens one by one gives (GPU against GPU):
    a chain of 7 in one pass vs seven N=1 passes that each commit their root."""
    cfg = gen.MODELS["tiny"]
    twin = Twin(cfg, 64, scale=4.0)
    prefix = gen.gen_prefix_tokens(cfg, 9)
    twin.v.prefill(0, torch.as_tensor(prefix, device=DEV))
    chain = gen.gen_tokens(cfg, 7, seed=5)
    one = twin.gpu_pass(9, chain, gen.tree_chain(7))
    for i, t in enumerate(chain):
        # N = 1: the root is always verified, so the pass commits it at slot 9 + i
        step = twin.gpu_pass(9 + i, [t], [-1])
        assert step["scalars"][B.S_NEW_PREFIX_LEN] == 10 + i
        scale = np.abs(one["logits"][i]).max()
        assert np.abs(step["logits"][0] - one["logits"][i]).max() <= 2e-5 * scale


# ----------------------------------------------------------------------------- bf16

def bf16_case(cfg, P, n, levels, branching, flags=0, seed=0, scale=1.0, max_seq=None):
    twin = Twin(cfg, max_seq or (P + n + 8), flags=flags, seed=seed, scale=scale)
    twin.fill_prefix_synthetic(P)
    parent = gen.tree_random(n, levels, branching, seed) if n > 1 else np.array([-1], np.int32)
    tokens = gen.gen_tokens(cfg, n, seed)
    return twin, parent, tokens


def run_bf16_parity(twin, P, parent, tokens, plant=True):
    cfg = twin.cfg
    before = twin.v.kv_view()[:, :, :, :P].clone()
    ref = twin.oracle_pass(P, tokens, parent)
    out = twin.gpu_pass(P, tokens, parent)
    logits_close(out["logits"], ref.logits, BF16_TOL)
    undecided = argmax_agrees_where_decided(out["argmax"], ref.logits, BF16_TOL)
    acc = check_acceptance_against_oracle(out, tokens, parent)
    assert torch.equal(twin.v.kv_view()[:, :, :, :P], before)
    if plant:
        # plant the GPU's own argmax so that both sides verify a real path, then freeze the tokens
        tok = tokens
        for it in range(4):
            tok = gen.plant_tokens(parent, tok, out["argmax"], seed=it, prob=0.9)
            out = twin.gpu_pass(P, tok, parent)
        ref = twin.oracle_pass(P, tok, parent)
        logits_close(out["logits"], ref.logits, BF16_TOL)
        argmax_agrees_where_decided(out["argmax"], ref.logits, BF16_TOL)
        acc = check_acceptance_against_oracle(out, tok, parent)
        # rolled-back rows: value-wise against the oracle's K/V of the verified nodes (bf16 storage)
        got = cache_rows(twin.v, P + acc.accepted_len)
        for l in range(cfg.n_layers):
            for which, tree in ((0, ref.tree_k[l]), (1, ref.tree_v[l])):
                want = tree[acc.path].reshape(acc.accepted_len, cfg.n_heads, cfg.head_dim).transpose(1, 0, 2)
                have = got[l, which, :, P:]
                assert np.abs(have - want).max() <= BF16_TOL * max(np.abs(want).max(), 1e-6)
    return undecided, acc


SMALL_BF16 = gen.ModelConfig("small-bf16", 2, 512, 4, 128, 1408, 2048, "bf16")


@pytest.mark.parametrize("flags", [B.FLAG_SIMT_GEMM | B.FLAG_SIMT_ATTN, B.FLAG_SIMT_ATTN, B.FLAG_SIMT_GEMM, 0])
@pytest.mark.parametrize("P,n", [(100, 20), (0, 1), (64, 128), (37, 33)])
def test_bf16_small_whole_pass(flags, P, n):
    twin, parent, tokens = bf16_case(SMALL_BF16, P, n, 10, "uniform4", flags=flags, seed=P + n, scale=3.0)
    run_bf16_parity(twin, P, parent, tokens)


def test_bf16_chain_equals_single_token_passes():
    twin, _, _ = bf16_case(SMALL_BF16, 50, 1, 1, "uniform4", seed=3, scale=3.0, max_seq=80)
    chain = gen.gen_tokens(SMALL_BF16, 6, seed=9)
    one = twin.gpu_pass(50, chain, gen.tree_chain(6))
    for i, t in enumerate(chain):
        step = twin.gpu_pass(50 + i, [t], [-1])
        scale = np.abs(one["logits"][i]).max()
        # same arithmetic up to accumulation order and the bf16 rounding of slightly different partial sums
        assert np.abs(step["logits"][0] - one["logits"][i]).max() <= BF16_TOL * scale


def test_sibling_isolation_bit_exact():
    """Changing the token of a node that is not on a node's root path leaves that node's logits
    bit-identical (the mask gives it weight exactly zero)."""
    twin, parent, tokens = bf16_case(SMALL_BF16, 70, 24, 6, "uniform4", seed=4, scale=3.0)
    a = twin.gpu_pass(70, tokens, parent)
    i = 23
    path = set()
    j = i
    while j >= 0:
        path.add(j); j = int(parent[j])
    other = [k for k in range(24) if k not in path][-1]
    t2 = tokens.copy(); t2[other] = (t2[other] + 1) % SMALL_BF16.vocab
    b = twin.gpu_pass(70, t2, parent)
    assert np.array_equal(a["logits"][i], b["logits"][i])
    assert not np.array_equal(a["logits"][other], b["logits"][other])


@pytest.mark.parametrize("name,layers", [("7b", 2), ("13b", 1)])
def test_full_width_truncated_depth(name, layers):
    """7B / 13B widths (all tile counts, k-splits and epilogues of the real shapes) with few
    layers, so that the oracle finishes in seconds."""
    w = gen.WORKLOADS["C2" if name == "7b" else "C3"]
    cfg = gen.shrink(gen.MODELS[name], layers)
    twin = Twin(cfg, w.prefix_len + w.n_nodes + 8, keep_host=True)
    twin.fill_prefix_synthetic(w.prefix_len)
    parent = gen.gen_tree(w)
    tokens = gen.gen_tokens(cfg, w.n_nodes)
    run_bf16_parity(twin, w.prefix_len, parent, tokens, plant=False)


# ----------------------------------------------------------------------------- errors and the host entry

def test_error_paths():
    cfg = SMALL_BF16
    twin = Twin(cfg, 64, scale=3.0)
    twin.fill_prefix_synthetic(10)
    before = twin.v.kv_view().clone()
    # malformed tree -> device status, cache untouched, nothing accepted
    out = twin.gpu_pass(10, [1, 2, 3], [-1, 2, 0])
    assert out["scalars"][B.S_STATUS] == B.ERR_BAD_TREE
    assert out["scalars"][B.S_ACCEPTED_LEN] == 0 and out["scalars"][B.S_NEW_PREFIX_LEN] == 10
    assert torch.equal(twin.v.kv_view()[:, :, :, :10], before[:, :, :, :10])
    # token out of range
    out = twin.gpu_pass(10, [1, cfg.vocab, 3], [-1, 0, 0])
    assert out["scalars"][B.S_STATUS] == B.ERR_BAD_TOKEN
    assert torch.equal(twin.v.kv_view()[:, :, :, :10], before[:, :, :, :10])
    # host-detected
    dev = twin.v.device
    t = torch.zeros(60, dtype=torch.int32, device=dev)
    with pytest.raises(B.LlmcadError) as e:
        twin.v.verify_tree(10, t, t)
    assert e.value.code == B.ERR_CAPACITY
    t = torch.zeros(129, dtype=torch.int32, device=dev)
    with pytest.raises(B.LlmcadError) as e:
        twin.v.verify_tree(0, t, t)
    assert e.value.code == B.ERR_UNSUPPORTED
    # the context still works afterwards
    out = twin.gpu_pass(10, [1, 2, 3], [-1, 0, 0])
    assert out["scalars"][B.S_STATUS] == 0 and out["scalars"][B.S_ACCEPTED_LEN] >= 1


def test_bounded_wait_runs_out_and_the_context_survives():
    """The failure path of the device-side waits: with the limit lowered to 1 ms, a GEMM whose
    activation copies are withheld (a launch flag, nothing faults) never sees its ring stages fill:
    every role gives up, the kernel reports TIMEOUT in the status word, frees its tensor memory and
    returns; the same context then runs a pass that is bit for bit what it produced before."""
    twin, parent, tokens = bf16_case(SMALL_BF16, 40, 20, 6, "uniform4", seed=8, scale=3.0)
    before = twin.gpu_pass(40, tokens, parent)
    assert before["scalars"][B.S_STATUS] == 0
    with pytest.raises(B.LlmcadError) as e:          # refuses to run with the default limit of 2 s
        twin.v.selftest_wait_timeout()
    assert e.value.code == B.ERR_INVALID_ARG
    twin.v.set_wait_limit_ns(1_000_000)
    import time
    t0 = time.perf_counter()
    assert twin.v.selftest_wait_timeout() == B.ERR_TIMEOUT
    assert time.perf_counter() - t0 < 1.0            # the kernel came back after ~1 ms + its 2 ms drain
    assert twin.v.selftest_wait_timeout() == B.ERR_TIMEOUT     # and again: nothing is left behind
    twin.v.set_wait_limit_ns(0)
    after = twin.gpu_pass(40, tokens, parent)
    assert after["scalars"][B.S_STATUS] == 0
    assert np.array_equal(after["logits"], before["logits"]) and np.array_equal(after["argmax"], before["argmax"])
    assert np.array_equal(after["scalars"], before["scalars"])


def test_host_entry_equals_device_entry():
    twin, parent, tokens = bf16_case(SMALL_BF16, 40, 20, 6, "uniform4", seed=8, scale=3.0)
    a = twin.gpu_pass(40, tokens, parent)
    n = len(tokens)
    host = {
        "logits": torch.empty((n, SMALL_BF16.vocab), dtype=torch.float32).pin_memory(),
        "argmax": torch.empty(n, dtype=torch.int32).pin_memory(),
        "accepted_path": torch.full((128,), -1, dtype=torch.int32).pin_memory(),
        "scalars": torch.zeros(8, dtype=torch.int32).pin_memory(),
    }
    th = torch.as_tensor(tokens).pin_memory()
    ph = torch.as_tensor(parent).pin_memory()
    twin.v.verify_tree_host(40, th, ph, host)
    assert np.array_equal(host["logits"].numpy(), a["logits"])
    assert np.array_equal(host["argmax"].numpy(), a["argmax"])
    assert np.array_equal(host["scalars"].numpy(), a["scalars"])
    L = a["scalars"][B.S_ACCEPTED_LEN]
    assert np.array_equal(host["accepted_path"].numpy()[:L], a["accepted_path"][:L])


# ----------------------------------------------------------------------------- tuning paths

_TUNING_SCRIPT = r"""
import sys, os
sys.path.insert(0, os.path.join(sys.argv[1], "tests")); sys.path.insert(0, sys.argv[1])
import numpy as np
import test_gpu_pass as T
twin, parent, tokens = T.bf16_case(T.SMALL_BF16, 100, 40, 10, "uniform4", seed=7, scale=3.0)
T.run_bf16_parity(twin, 100, parent, tokens)
twin, parent, tokens = T.bf16_case(T.SMALL_BF16, 64, 128, 12, "uniform4", seed=8, scale=3.0)
T.run_bf16_parity(twin, 64, parent, tokens, plant=False)
print("ok")
"""


@pytest.mark.parametrize("env", [{"LLMCAD_PDL": "0"}, {"LLMCAD_SYNC_COUNTERS": "1"}, {"LLMCAD_COMP": "0"},
                                 {"LLMCAD_GEMM_PAIR_K": "1"}, {"LLMCAD_GEMM_STAGES": "2"},
                                 {"LLMCAD_ATTN_T5_MIN_N": "1"}, {"LLMCAD_ATTN_T5_MIN_N": "0"}])
def test_tuning_paths_stay_correct(env):
    """The environment knobs select other code paths of the same kernels (no programmatic dependent
    launch, hand-over between kernels through completion counters, plain bf16 activations, ring items
    of one k-block, a two-stage ring, the tcgen05 attention kernel for every tree size, the mma.sync
    attention kernel for every tree size): each must still match the oracle. The knobs are read once per
    process, hence the child process."""
    import os, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    e = dict(os.environ, **env)
    r = subprocess.run([sys.executable, "-c", _TUNING_SCRIPT, root], env=e, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stdout[-2000:] + r.stderr[-4000:]


def test_debug_build_with_device_side_checks_finds_nothing():
    """The library built with -DLLMCAD_CHECKS verifies, on the device, the indices it derives from data
    and from the launch arithmetic (workspace slots, cache slots, path entries) and reports a failed
    check through the status word instead of touching memory. The same parity cases must pass under it
    with status 0: the stand-in for a memory checker on a machine that has none."""
    import os, subprocess, sys
    from paper_2309_04255_b200 import build as libbuild
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    e = dict(os.environ, LLMCAD_LIB=libbuild.build(checks=True))
    r = subprocess.run([sys.executable, "-c", _TUNING_SCRIPT, root], env=e, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stdout[-2000:] + r.stderr[-4000:]


def test_queued_passes_of_changing_size_are_reproducible():
    """Passes over trees of different sizes queued back to back on one stream (no host
    synchronisation in between) must each give, bit for bit, what the same pass gives alone: the
    arrival counters, the alternating counter sets and the helpers' flags of the GEMM tail leave no
    state behind that depends on timing or on the previous launch's shape."""
    cfg = gen.shrink(gen.MODELS["7b"], 2)
    P = 200
    twin = Twin(cfg, P + 136, keep_host=False)
    twin.fill_prefix_synthetic(P)
    v = twin.v
    cases = []
    for n in (1, 16, 32, 64, 128):
        tokens = torch.as_tensor(gen.gen_tokens(cfg, n, seed=n), device=DEV)
        parent = torch.as_tensor(gen.tree_random(n, 12, "uniform4", n) if n > 1 else np.array([-1], np.int32), device=DEV)
        out = v.verify_tree(P, tokens, parent)
        torch.cuda.synchronize()
        assert out["scalars"][B.S_STATUS].item() == 0
        cases.append((n, tokens, parent, {k: t.clone() for k, t in out.items()}))
    rng = np.random.default_rng(1)
    for _ in range(4):
        outs = []
        for _ in range(40):
            ci = int(rng.integers(len(cases)))
            n, tokens, parent, _ref = cases[ci]
            o = v.new_outputs(n)
            v.verify_tree(P, tokens, parent, out=o)
            outs.append((ci, o))
        torch.cuda.synchronize()
        for ci, o in outs:
            ref = cases[ci][3]
            assert torch.equal(o["logits"], ref["logits"]) and torch.equal(o["argmax"], ref["argmax"])
            assert torch.equal(o["scalars"], ref["scalars"]) and torch.equal(o["accepted_path"], ref["accepted_path"])
