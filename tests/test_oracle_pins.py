"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test names the statement it pins. The library implementation used as an outside
opinion of the decoder is transformers' LlamaForCausalLM (fp64, CPU, eager attention).
"""
import os

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2309_04255_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
HF_TOL = 2e-5  # the library decoder evaluates its norms and rotary table in fp32 even when cast to fp64


# ----------------------------------------------------------------------------- helpers

def pin_model(seed=0, n_layers=2, d=32, H=4, hd=8, f=48, V=64):
    """A small model with weights large enough that softmax, SiLU and the norms are far
    from their linear regime, and with random norm gains."""
    cfg = gen.ModelConfig("pin", n_layers, d, H, hd, f, V, "f32")
    g = np.random.default_rng(1000 + seed)

    def w(*shape, s):
        return torch.from_numpy((g.standard_normal(shape) * s).astype(np.float32))

    glob = {"tok_embed": w(V, d, s=1.0), "final_norm": w(d, s=0.3) + 1.0, "lm_head": w(V, d, s=0.5)}
    layers = []
    for _ in range(n_layers):
        layers.append({
            "attn_norm": w(d, s=0.3) + 1.0, "wq": w(d, d, s=0.5), "wk": w(d, d, s=0.5), "wv": w(d, d, s=0.4),
            "wo": w(d, d, s=0.3), "ffn_norm": w(d, s=0.3) + 1.0, "w_gate": w(f, d, s=0.4), "w_up": w(f, d, s=0.4),
            "w_down": w(d, f, s=0.3)})
    return cfg, glob, layers


def to_half_split(W, H, hd):
    """Row permutation that maps rotary on interleaved pairs (2t, 2t+1) to rotary on
    split halves (t, t + hd/2), the convention of the library decoder."""
    d_in = W.shape[1]
    return W.reshape(H, hd // 2, 2, d_in).permute(0, 2, 1, 3).reshape(H * hd, d_in)


_hf_cache = {}


def hf_model(cfg, glob, layers, key):
    if key in _hf_cache:
        return _hf_cache[key]
    from transformers import LlamaConfig, LlamaForCausalLM
    hc = LlamaConfig(vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.d_ffn,
                     num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
                     num_key_value_heads=cfg.n_heads, head_dim=cfg.head_dim, max_position_embeddings=512,
                     rms_norm_eps=cfg.rms_eps, rope_theta=cfg.rope_base, attention_bias=False,
                     mlp_bias=False, tie_word_embeddings=False, attn_implementation="eager")
    m = LlamaForCausalLM(hc).double().eval()
    sd = {"model.embed_tokens.weight": glob["tok_embed"], "model.norm.weight": glob["final_norm"],
          "lm_head.weight": glob["lm_head"]}
    for l, w in enumerate(layers):
        p = f"model.layers.{l}."
        sd[p + "self_attn.q_proj.weight"] = to_half_split(w["wq"], cfg.n_heads, cfg.head_dim)
        sd[p + "self_attn.k_proj.weight"] = to_half_split(w["wk"], cfg.n_heads, cfg.head_dim)
        sd[p + "self_attn.v_proj.weight"] = w["wv"]
        sd[p + "self_attn.o_proj.weight"] = w["wo"]
        sd[p + "mlp.gate_proj.weight"] = w["w_gate"]
        sd[p + "mlp.up_proj.weight"] = w["w_up"]
        sd[p + "mlp.down_proj.weight"] = w["w_down"]
        sd[p + "input_layernorm.weight"] = w["attn_norm"]
        sd[p + "post_attention_layernorm.weight"] = w["ffn_norm"]
    missing, unexpected = m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing if "rotary" not in k], missing
    assert not unexpected
    _hf_cache[key] = m
    return m


def hf_logits(m, seq):
    with torch.no_grad():
        return m(torch.tensor([list(map(int, seq))])).logits[0].numpy()


def prefill_oracle(cfg, glob, layers, prefix_tokens, max_seq=128):
    dec = orc.SequentialDecoder(cfg, glob, layers, max_seq)
    last = None
    for t in prefix_tokens:
        last = dec.step(int(t))
    return dec, last


def run_tree(cfg, glob, layers, dec, P, tokens, parent):
    return orc.verify_tree(cfg, glob, lambda l: layers[l], lambda l: dec.cache_heads(l, P), P, tokens, parent)


def path_of(parent, i):
    p = []
    while i >= 0:
        p.append(i)
        i = int(parent[i])
    return p[::-1]


def read_golden(name):
    blocks = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":")
            blocks.append((k.strip(), [int(t) for t in v.split()]))
    return blocks


# ----------------------------------------------------------------------------- mask table

def test_mask_paper_example():
    """Sec. 3.2 tree decoder: the step producing "7" sees positions 1,2,3,5 only."""
    items = read_golden("mask_example.txt")
    parent = dict(items)["parent_idx"]
    st, depth, pos, anc = orc.tree_prep(parent, 10)
    assert st == 0
    queries = [(v[0], items[i + 1][1]) for i, (k, v) in enumerate(items) if k == "query"]
    assert len(queries) == 2
    for q, visible in queries:
        assert sorted(np.nonzero(anc[q])[0].tolist()) == visible
    assert depth.tolist() == [0, 1, 2, 3, 3, 4, 4]
    assert pos.tolist() == [10 + x for x in depth.tolist()]


@pytest.mark.parametrize("seed", range(6))
def test_mask_invariants(seed):
    parent = gen.tree_random(40, 9, "uniform4", seed)
    st, depth, pos, anc = orc.tree_prep(parent, 7)
    assert st == 0
    for i in range(len(parent)):
        assert anc[i].sum() == depth[i] + 1          # one bit per level of the branch
        assert anc[i, i] == 1
        assert anc[i, i + 1:].sum() == 0             # nothing later than the node itself
        # brute force: walk to the root
        assert sorted(path_of(parent, i)) == np.nonzero(anc[i])[0].tolist()
        if parent[i] >= 0:
            rest = anc[i].copy(); rest[i] = 0
            assert (rest == anc[parent[i]]).all()
    assert (pos == 7 + depth).all()


def test_bad_trees_rejected():
    for bad in ([0, 0, 1], [-1, -1, 0], [-1, 1, 0], [-1, 0, 3], [-1, 5]):
        st, *_ = orc.tree_prep(bad, 0)
        assert st == 1, bad


# ----------------------------------------------------------------------------- closed forms of the steps

def test_linear_matches_library_matmul():
    g = np.random.default_rng(0)
    W = g.standard_normal((37, 53)).astype(np.float32)
    x = g.standard_normal((5, 53))
    np.testing.assert_allclose(orc.linear(W, x), x @ W.astype(np.float64).T, rtol=1e-13, atol=1e-13)
    # a transposed operand or swapped dims would fail this non-square case


def test_rmsnorm_closed_form_and_library():
    d = 48
    g = np.random.default_rng(1).standard_normal(d).astype(np.float32)
    for c in (0.5, -3.0):
        out = orc.rmsnorm(np.full((1, d), c), g, 1e-5)
        np.testing.assert_allclose(out[0], g.astype(np.float64) * c / np.sqrt(c * c + 1e-5), rtol=1e-13)
    x = np.random.default_rng(2).standard_normal((3, d))
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (d,), torch.from_numpy(g).double(), 1e-5).numpy()
    np.testing.assert_allclose(orc.rmsnorm(x, g, 1e-5), ref, rtol=1e-12, atol=1e-14)
    # eps matters: with x = 0 the output is 0, not NaN
    assert np.all(orc.rmsnorm(np.zeros((1, d)), g, 1e-5) == 0)


def test_rope_closed_forms():
    H, hd = 2, 8
    g = np.random.default_rng(3)
    v = g.standard_normal((4, H * hd))
    # position 0 is the identity
    np.testing.assert_array_equal(orc.rope(v, [0, 0, 0, 0], H, hd, 10000.0), v)
    # rotations preserve the norm of every pair
    r = orc.rope(v, [1, 17, 300, 4095], H, hd, 10000.0)
    np.testing.assert_allclose((r.reshape(4, H, hd // 2, 2) ** 2).sum(-1), (v.reshape(4, H, hd // 2, 2) ** 2).sum(-1), rtol=1e-12)
    # unit vector on pair t rotates to (cos, sin) of pos * base^(-2t/hd)
    for t in range(hd // 2):
        e = np.zeros((1, H * hd)); e[0, 2 * t] = 1.0
        out = orc.rope(e, [5], H, hd, 10000.0)
        ang = 5 * 10000.0 ** (-2.0 * t / hd)
        np.testing.assert_allclose(out[0, 2 * t: 2 * t + 2], [np.cos(ang), np.sin(ang)], rtol=1e-12, atol=1e-15)
        assert np.count_nonzero(out) <= 2
    # relative-position property: <rope(q,m), rope(k,n)> depends on m-n only
    q = g.standard_normal((1, H * hd)); k = g.standard_normal((1, H * hd))
    a = (orc.rope(q, [9], H, hd, 10000.0) * orc.rope(k, [4], H, hd, 10000.0)).sum()
    b = (orc.rope(q, [105], H, hd, 10000.0) * orc.rope(k, [100], H, hd, 10000.0)).sum()
    np.testing.assert_allclose(a, b, rtol=1e-10)


def test_attention_closed_forms():
    H, hd = 2, 4
    g = np.random.default_rng(4)
    # P = 0, a single root: the only visible key is the node itself -> output = its V row exactly
    q = g.standard_normal((1, H * hd)); k = g.standard_normal((1, H * hd)); v = g.standard_normal((1, H * hd))
    o = orc.tree_attention(q, np.zeros((H, 0, hd)), np.zeros((H, 0, hd)), k, v, np.ones((1, 1)), H, hd)
    np.testing.assert_allclose(o, v, rtol=1e-15)
    # all keys equal -> uniform weights -> mean of visible V rows
    P, n = 3, 3
    parent = [-1, 0, 0]
    _, _, _, anc = orc.tree_prep(parent, P)
    kk = np.tile(g.standard_normal((1, 1, hd)), (H, P, 1))
    tk = np.tile(kk[:, 0, :].reshape(1, H * hd), (n, 1))
    pv = g.standard_normal((H, P, hd)); tv = g.standard_normal((n, H * hd))
    o = orc.tree_attention(g.standard_normal((n, H * hd)), kk, pv, tk, tv, anc, H, hd)
    for i, vis in enumerate(([0], [0, 1], [0, 2])):
        for h in range(H):
            rows = np.concatenate([pv[h], tv[vis].reshape(len(vis), H, hd)[:, h]], 0)
            np.testing.assert_allclose(o[i, h * hd:(h + 1) * hd], rows.mean(0), rtol=1e-12)
    # against the library softmax attention with an explicit boolean mask
    P, n = 5, 6
    parent = gen.tree_random(n, 4, "uniform4", 1)
    _, _, _, anc = orc.tree_prep(parent, P)
    q = g.standard_normal((n, H * hd)); pk = g.standard_normal((H, P, hd)); pv = g.standard_normal((H, P, hd))
    tk = g.standard_normal((n, H * hd)); tv = g.standard_normal((n, H * hd))
    o = orc.tree_attention(q, pk, pv, tk, tv, anc, H, hd)
    K = torch.cat([torch.from_numpy(pk), torch.from_numpy(tk).reshape(n, H, hd).permute(1, 0, 2)], 1)
    Vv = torch.cat([torch.from_numpy(pv), torch.from_numpy(tv).reshape(n, H, hd).permute(1, 0, 2)], 1)
    mask = torch.cat([torch.ones(n, P, dtype=torch.bool), torch.from_numpy(anc.astype(bool))], 1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).reshape(n, H, hd).permute(1, 0, 2)[None], K[None], Vv[None], attn_mask=mask[None, None])
    np.testing.assert_allclose(o, ref[0].permute(1, 0, 2).reshape(n, H * hd).numpy(), rtol=1e-11, atol=1e-13)


def test_zero_layer_pass_is_a_matmul():
    """With no decoder layers the pass is argmax(norm(E[tok]) W_lm^T)."""
    cfg, glob, _ = pin_model(5, n_layers=0)
    tokens = [3, 9, 9, 60]
    res = orc.verify_tree(cfg, glob, None, None, 0, tokens, [-1, 0, 0, 1])
    E = glob["tok_embed"].double()[tokens]
    xn = torch.nn.functional.rms_norm(E, (cfg.d_model,), glob["final_norm"].double(), cfg.rms_eps)
    ref = (xn @ glob["lm_head"].double().T).numpy()
    np.testing.assert_allclose(res.logits, ref, rtol=1e-12, atol=1e-13)
    assert (res.argmax == ref.argmax(1)).all()
    # nodes holding the same token see the same logits (no positions, no attention)
    np.testing.assert_array_equal(res.logits[1], res.logits[2])


def test_argmax_ties_lowest_index():
    lg = np.zeros((2, 7)); lg[0, [2, 5]] = 3.0; lg[1, :] = -1.0
    assert orc.argmax(lg).tolist() == [2, 0]


# ----------------------------------------------------------------------------- the decoder against a library

def test_sequential_decoder_matches_library_llama():
    """Pins RMSNorm/eps, rotary pairing (through the standard row permutation), the
    1/sqrt(hd) scale, SwiGLU and the residual layout of sequential.c."""
    cfg, glob, layers = pin_model(0)
    m = hf_model(cfg, glob, layers, 0)
    seq = gen.gen_tokens(cfg, 11, seed=3)
    ref = hf_logits(m, seq)
    dec = orc.SequentialDecoder(cfg, glob, layers, 32)
    for t, tok in enumerate(seq):
        np.testing.assert_allclose(dec.step(int(tok)), ref[t], rtol=HF_TOL, atol=HF_TOL * np.abs(ref).max())
    assert np.abs(ref).max() > 1.0  # not a near-zero regime


def test_chain_tree_equals_sequential_decoding():
    """Sec. 3.2: examining N tokens in one shot gives the same results as examining
    them sequentially. Chain tree, with and without a prefix."""
    cfg, glob, layers = pin_model(1)
    for P in (0, 6):
        prefix = gen.gen_prefix_tokens(cfg, P, seed=1)
        chain = gen.gen_tokens(cfg, 7, seed=2)
        dec, _ = prefill_oracle(cfg, glob, layers, prefix)
        res = run_tree(cfg, glob, layers, dec, P, chain, gen.tree_chain(7))
        for i, tok in enumerate(chain):
            np.testing.assert_allclose(res.logits[i], dec.step(int(tok)), rtol=1e-10, atol=1e-11)
        # the tree pass's K/V rows are what sequential decoding cached at the same positions
        for l in range(cfg.n_layers):
            np.testing.assert_allclose(res.tree_k[l], dec.kc[l, P:P + 7], rtol=1e-10, atol=1e-12)
            np.testing.assert_allclose(res.tree_v[l], dec.vc[l, P:P + 7], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("seed,shape", [(0, "binary"), (1, "uniform4"), (2, "geometric4"), (3, "star")])
def test_every_node_equals_its_path_run_as_a_sequence(seed, shape):
    """Brute force on tiny trees: node i's logits are those of the library decoder run
    on prefix + tokens of the root-to-i path, last position."""
    cfg, glob, layers = pin_model(2)
    m = hf_model(cfg, glob, layers, 2)
    P = 5
    prefix = gen.gen_prefix_tokens(cfg, P, seed=seed)
    if shape == "binary":
        parent = gen.tree_binary(4)
    elif shape == "star":
        parent = gen.tree_star(6)
    else:
        parent = gen.tree_random(14, 5, shape, seed)
    tokens = gen.gen_tokens(cfg, len(parent), seed=seed)
    dec, _ = prefill_oracle(cfg, glob, layers, prefix)
    res = run_tree(cfg, glob, layers, dec, P, tokens, parent)
    for i in range(len(parent)):
        seq = list(prefix) + [tokens[j] for j in path_of(parent, i)]
        ref = hf_logits(m, seq)[-1]
        np.testing.assert_allclose(res.logits[i], ref, rtol=HF_TOL, atol=HF_TOL * np.abs(ref).max())


def test_relabelling_and_sibling_isolation():
    cfg, glob, layers = pin_model(3)
    P = 4
    prefix = gen.gen_prefix_tokens(cfg, P, seed=7)
    parent = gen.tree_random(12, 5, "uniform4", 7)
    tokens = gen.gen_tokens(cfg, 12, seed=7)
    dec, _ = prefill_oracle(cfg, glob, layers, prefix)
    res = run_tree(cfg, glob, layers, dec, P, tokens, parent)
    newp, perm = gen.relabel_tree(parent, 5)
    assert not (perm == np.arange(12)).all()
    res2 = run_tree(cfg, glob, layers, dec, P, tokens[perm], newp)
    np.testing.assert_allclose(res2.logits, res.logits[perm], rtol=1e-12, atol=1e-13)
    # changing a non-ancestor's token leaves a node's logits bit-identical
    i = 11
    anc = set(path_of(parent, i))
    other = [j for j in range(12) if j not in anc][0]
    t2 = tokens.copy(); t2[other] = (t2[other] + 1) % cfg.vocab
    res3 = run_tree(cfg, glob, layers, dec, P, t2, parent)
    np.testing.assert_array_equal(res3.logits[i], res.logits[i])
    assert not np.array_equal(res3.logits[other], res.logits[other])


# ----------------------------------------------------------------------------- acceptance

def test_acceptance_paper_example():
    g = dict(read_golden("acceptance_example.txt"))
    acc = orc.accept(g["parent_idx"], g["tokens"], g["argmax"])
    assert acc.path.tolist() == g["path"]
    assert acc.next_token == g["next_token"][0]
    assert acc.rectified == g["rectified"][0]
    assert [g["tokens"][i] for i in acc.path] + [acc.next_token] == g["verified_tokens"]
    assert acc.accepted_len == 3 and acc.n_correct == 2
    assert acc.n_all == 3          # branch 1,2,5,7 through the last verified node: 3 draft tokens after the root


def brute_accept(parent, tokens, amax):
    """Enumerate every root-to-node path; a path is correct when each of its draft
    tokens equals the target's output at the node before it; take the longest,
    ties to the lowest end node."""
    best = None
    for i in range(len(parent)):
        p = path_of(parent, i)
        ok = all(tokens[p[j + 1]] == amax[p[j]] for j in range(len(p) - 1))
        if ok and (best is None or len(p) > len(best)):
            best = p
    return best


@pytest.mark.parametrize("seed", range(20))
def test_acceptance_brute_force_random(seed):
    g = np.random.default_rng(seed)
    n = int(g.integers(1, 25))
    parent = gen.tree_random(n, 6, "uniform4", seed) if n > 1 else np.array([-1], np.int32)
    V = 3  # tiny vocabulary: many matches, duplicate sibling tokens included
    tokens = g.integers(0, V, n); amax = g.integers(0, V, n)
    acc = orc.accept(parent, tokens, amax)
    best = brute_accept(parent, tokens, amax)
    assert acc.path.tolist() == best
    assert acc.accepted_len == len(best) and acc.next_token == amax[best[-1]]
    has_child = any(parent[c] == best[-1] for c in range(n))
    assert acc.rectified == int(has_child)
    # n_all: longest draft branch through the last verified node, root excluded
    deepest = max(len(path_of(parent, j)) - 1 for j in range(n) if best[-1] in path_of(parent, j))
    assert acc.n_all == deepest and acc.n_correct == len(best) - 1


def test_acceptance_equals_sequential_greedy_check_and_compaction():
    """The verified sequence is what sequential greedy decoding of the target produces,
    and the rolled-back cache is the cache of prefix + verified tokens."""
    cfg, glob, layers = pin_model(4)
    P = 5
    prefix = gen.gen_prefix_tokens(cfg, P, seed=11)
    parent = gen.tree_random(16, 6, "uniform4", 11)
    tokens = gen.gen_tokens(cfg, 16, seed=11)
    dec, _ = prefill_oracle(cfg, glob, layers, prefix)
    # plant the target's own outputs (taken from a first oracle pass) along some branches
    first = run_tree(cfg, glob, layers, dec, P, tokens, parent)
    for it in range(6):  # iterate: planting a child changes its descendants' context
        tokens = gen.plant_tokens(parent, tokens, first.argmax, seed=it, prob=0.9)
        first = run_tree(cfg, glob, layers, dec, P, tokens, parent)
    res = first
    acc = res.acceptance
    assert acc.accepted_len >= 3, "planting should give a non-trivial verified sequence"
    # sequential greedy check
    dec.truncate(P)
    tok = int(tokens[0])
    greedy = []
    for _ in range(acc.accepted_len):
        tok = int(np.argmax(dec.step(tok)))
        greedy.append(tok)
    assert [int(tokens[i]) for i in acc.path[1:]] + [acc.next_token] == greedy
    kids = [int(tokens[c]) for c in range(16) if parent[c] == acc.path[-1]]
    assert acc.next_token not in kids
    # compaction == cache after consuming prefix + verified tokens
    for l in range(cfg.n_layers):
        pk, pv = dec.cache_heads(l, P)
        newk = orc.compact(pk, res.tree_k[l], acc.path, cfg.n_heads, cfg.head_dim)
        newv = orc.compact(pv, res.tree_v[l], acc.path, cfg.n_heads, cfg.head_dim)
        refk, refv = dec.cache_heads(l, P + acc.accepted_len)
        np.testing.assert_allclose(newk, refk, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(newv, refv, rtol=1e-10, atol=1e-12)
    assert res.new_prefix_len == P + acc.accepted_len


def test_tiny_config_whole_pass_against_library():
    """Config 1 (2 layers, d 256, 4x64 heads, FFN 688, vocab 1024, prefix 32, full
    binary tree of 15 nodes) through the oracle and through the library decoder."""
    cfg = gen.MODELS["tiny"]
    glob = gen.gen_globals(cfg)
    layers = [gen.gen_layer(cfg, l) for l in range(cfg.n_layers)]
    m = hf_model(cfg, glob, layers, "tiny")
    w = gen.WORKLOADS["C1"]
    prefix = gen.gen_prefix_tokens(cfg, w.prefix_len)
    parent = gen.gen_tree(w)
    tokens = gen.gen_tokens(cfg, w.n_nodes)
    dec, _ = prefill_oracle(cfg, glob, layers, prefix)
    res = run_tree(cfg, glob, layers, dec, w.prefix_len, tokens, parent)
    for i in (0, 3, 7, 14):
        seq = list(prefix) + [tokens[j] for j in path_of(parent, i)]
        ref = hf_logits(m, seq)[-1]
        np.testing.assert_allclose(res.logits[i], ref, rtol=HF_TOL, atol=HF_TOL * np.abs(ref).max())


# ------------------------------------------------------------------ fallback scalars (Sec. 3.3, Eq. 3)

def test_alpha_update_closed_forms():
    """The two branches of Eq. 3 on values that can be checked by hand."""
    a = 0.01                                               # the paper's default threshold
    assert orc.alpha_update(a, 5, 5, 0.3) == a * 0.5       # no error: halved, whatever T_c
    # one of two draft tokens wrong, T_c = 1/4: alpha / (1/4)^(1/2) = 2 alpha
    assert abs(orc.alpha_update(a, 1, 2, 0.25) - 2 * a) < 1e-15
    # all wrong: alpha / T_c
    assert abs(orc.alpha_update(a, 0, 4, 0.125) - a / 0.125) < 1e-15
    # three of four wrong, T_c = 1/16: exponent 3/4 -> 16^(3/4) = 8
    assert abs(orc.alpha_update(a, 1, 4, 1.0 / 16) - 8 * a) < 1e-14
    # a fully confident tree does not move the threshold when there are errors
    assert orc.alpha_update(a, 2, 7, 1.0) == a
    # nothing verified
    assert orc.alpha_update(a, 0, 0, 0.5) == a


def test_alpha_update_monotonic():
    """With errors the threshold never drops, and it grows with the share of wrong tokens and with
    lower confidence; a run of k verifications without error divides it by 2^k."""
    a = 0.01
    prev = a
    for wrong in range(1, 9):
        cur = orc.alpha_update(a, 8 - wrong, 8, 0.4)
        assert cur > prev
        prev = cur
    assert orc.alpha_update(a, 3, 8, 0.2) > orc.alpha_update(a, 3, 8, 0.6) > a
    x = a
    for _ in range(6):
        x = orc.alpha_update(x, 4, 4, 0.9)
    assert x == a / 64


def test_tree_confidence_is_the_maximum():
    rng = np.random.default_rng(5)
    c = rng.uniform(0.01, 1.0, 17)
    assert orc.tree_confidence(c) == c.max()
    assert orc.tree_confidence([0.3]) == 0.3


# ------------------------------------------------------------------ confidences of the generating side

def test_topk_softmax_against_library_and_closed_forms():
    rng = np.random.default_rng(3)
    lg = rng.normal(0, 2, (5, 97))
    ids, probs = orc.topk_softmax(lg, 6)
    ref = torch.softmax(torch.from_numpy(lg), dim=-1).numpy()
    order = np.argsort(-lg, axis=1, kind="stable")[:, :6]
    assert np.array_equal(ids, order)
    np.testing.assert_allclose(probs, np.take_along_axis(ref, order, 1), rtol=1e-12)
    # equal logits: uniform probabilities, the lowest ids first
    ids, probs = orc.topk_softmax(np.zeros((1, 10)), 3)
    assert ids.tolist() == [[0, 1, 2]] and np.allclose(probs, 0.1)
    # two-token vocabulary: the logistic function
    ids, probs = orc.topk_softmax(np.array([[0.0, np.log(3.0)]]), 2)
    assert ids.tolist() == [[1, 0]] and np.allclose(probs, [[0.75, 0.25]])
    # all of the vocabulary: the probabilities add up to one and come in descending order
    ids, probs = orc.topk_softmax(lg[:1], 97)
    assert abs(probs.sum() - 1.0) < 1e-12 and np.all(np.diff(probs[0]) <= 0) and sorted(ids[0]) == list(range(97))
    # shift invariance, and no overflow on large logits
    a = orc.topk_softmax(lg, 4)[1]
    b = orc.topk_softmax(lg + 1000.0, 4)[1]
    np.testing.assert_allclose(a, b, rtol=1e-9)


def test_tree_branches_on_trees_with_known_branches():
    """Sec. 3.2: a branch per leaf, cumulative confidence = product over its draft tokens."""
    conf = np.array([0.123, 0.9, 0.8, 0.5, 0.25])          # the root's entry must not matter
    # chain root-1-2-3-4: one branch through everything
    leaf, cum, length = orc.tree_branches([-1, 0, 1, 2, 3], conf)
    assert leaf.tolist() == [4] and length.tolist() == [4]
    assert cum[0] == pytest.approx(0.9 * 0.8 * 0.5 * 0.25, rel=1e-15)
    # star: every child of the root is a branch of one token
    leaf, cum, length = orc.tree_branches([-1, 0, 0, 0, 0], conf)
    assert leaf.tolist() == [1, 2, 3, 4] and length.tolist() == [1, 1, 1, 1] and cum.tolist() == conf[1:].tolist()
    # root alone: one branch without draft tokens, confidence of the empty product
    leaf, cum, length = orc.tree_branches([-1], conf[:1])
    assert leaf.tolist() == [0] and length.tolist() == [0] and cum.tolist() == [1.0]
    # the tree of the verification figure's shape: 0 -> (1 -> (3, 4), 2 -> 5)
    leaf, cum, length = orc.tree_branches([-1, 0, 0, 1, 1, 2], np.array([1.0, 0.5, 0.4, 0.3, 0.2, 0.1]))
    assert leaf.tolist() == [3, 4, 5] and length.tolist() == [2, 2, 2]
    np.testing.assert_allclose(cum, [0.15, 0.10, 0.04], rtol=1e-15)


def test_tree_branches_against_path_walking():
    rng = np.random.default_rng(11)
    for n in (2, 7, 33, 128):
        parent = np.array(gen.tree_random(n, 10, "uniform4", n), dtype=np.int64)
        conf = rng.uniform(0.05, 1.0, n)
        leaf, cum, length = orc.tree_branches(parent, conf)
        children = {i: [j for j in range(n) if parent[j] == i] for i in range(n)}
        want = [i for i in range(n) if not children[i]]
        assert leaf.tolist() == want
        for b, i in enumerate(want):
            path = []
            while parent[i] >= 0:
                path.append(i)
                i = int(parent[i])
            assert length[b] == len(path)
            assert cum[b] == pytest.approx(float(np.prod(conf[path])) if path else 1.0, rel=1e-12)


def test_branch_pacer_closed_forms():
    """Eq. 1: f(x) = M C_x / sum C - T_x on values that can be checked by hand."""
    f, nxt = orc.branch_pacer([0.75, 0.25], [4, 4], 8)
    assert f.tolist() == [2.0, -2.0] and nxt == 0           # shares 6 and 2 of 8 tokens, each holds 4
    f, nxt = orc.branch_pacer([0.75, 0.25], [7, 1], 8)
    assert f.tolist() == [-1.0, 1.0] and nxt == 1           # the confident branch ran ahead of its share
    # equal confidences: everybody is entitled to M / N, the shortest branch goes next
    f, nxt = orc.branch_pacer([0.3] * 4, [3, 1, 2, 1], 10)
    np.testing.assert_allclose(f, [-0.5, 1.5, 0.5, 1.5], rtol=1e-15)
    assert nxt == 1                                         # tie between 1 and 3: the lower index
    # one branch: it owns every token
    f, nxt = orc.branch_pacer([0.01], [5], 9)
    assert f.tolist() == [4.0] and nxt == 0


def test_branch_pacer_invariants_and_max_min_choice():
    """sum_x f(x) = M - sum_x T_x; f only depends on confidence ratios; and the branch it picks is
    the one that leaves the smallest f largest after receiving a token (max-min fairness, Eq. 2),
    found here by trying every branch."""
    rng = np.random.default_rng(12)
    for n in (2, 3, 8, 31):
        c = rng.uniform(1e-4, 1.0, n) ** 3
        t = rng.integers(0, 12, n)
        m = float(t.sum() + rng.integers(0, 5))
        f, nxt = orc.branch_pacer(c, t, m)
        assert f.sum() == pytest.approx(m - t.sum(), abs=1e-9)
        f2, nxt2 = orc.branch_pacer(c * 0.37, t, m)
        np.testing.assert_allclose(f2, f, rtol=1e-12, atol=1e-12)
        assert nxt2 == nxt
        share = m * c / c.sum()
        np.testing.assert_allclose(f, share - t, rtol=1e-12, atol=1e-12)
        best = None
        for y in range(n):
            t_after = t.copy()
            t_after[y] += 1
            worst = (share - t_after).min()
            if best is None or worst > best[0] + 1e-12:
                best = (worst, y)
        # several branches can leave the same minimum; the chosen one must be among the best
        t_after = t.copy()
        t_after[nxt] += 1
        assert (share - t_after).min() == pytest.approx(best[0], abs=1e-9)
        assert f[nxt] == f.max()


# ----------------------------------------------------------------------------- INT4 weights (Sec. 4.1)

def test_int4_quantisation_hand_computed_groups():
    """Groups worked out by hand: the scale is the smallest power of two with max|w| <= 7 * 2^e, codes
    are w / 2^e rounded to nearest (halves to even) and clamped to [-8, 7]."""
    g = 4
    w = np.array([[0.7, -0.35, 0.0625, 0.0,          # max 0.7: 7 * 2^-4 = 0.4375 < 0.7 <= 7 * 2^-3 = 0.875 -> e = -3
                   7.0, -7.0, 3.5, 2.5,              # max 7 = 7 * 2^0 -> e = 0; 3.5 -> 4 (half to even), 2.5 -> 2
                   0.0, 0.0, 0.0, 0.0,               # all zero -> e = -126, codes 0
                   -8.0, 1.0, 0.5, -0.5]],           # max 8 > 7 -> e = 1: -8/2 = -4, 1/2 = 0.5 -> 0, 0.25 -> 0, -0.25 -> 0
                 np.float32)
    q, e = orc.quantize_int4(w, g)
    assert e.tolist() == [[-3, 0, -126, 1]]
    assert q.tolist() == [[6, -3, 0, 0, 7, -7, 4, 2, 0, 0, 0, 0, -4, 0, 0, 0]]     # 0.7/0.125 = 5.6 -> 6; -2.8 -> -3; 0.5 -> 0
    d = orc.dequantize_int4(q, e, g)
    assert d.tolist() == [[0.75, -0.375, 0.0, 0.0, 7.0, -7.0, 4.0, 2.0, 0.0, 0.0, 0.0, 0.0, -8.0, 0.0, 0.0, 0.0]]


def test_int4_quantisation_invariants():
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((37, 256)) * 0.02).astype(np.float32)
    w[3, 64:128] = 0.0
    w[5, 0] = 1.5                                    # an outlier sets its group's scale
    q, e = orc.quantize_int4(w)
    d = orc.dequantize_int4(q, e)
    assert q.min() >= -8 and q.max() <= 7
    scale = np.exp2(e.astype(np.float64)).repeat(64, axis=1)
    # nearest code: the error is at most half a step (the largest magnitude is at most 7 steps, so nothing clips)
    assert (np.abs(d.astype(np.float64) - w) <= 0.5 * scale + 1e-12).all()
    # the scale is the smallest admissible power of two: the group's largest magnitude exceeds 7 steps of the next smaller one
    gmax = np.abs(w).reshape(37, 4, 64).max(axis=2)
    nz = gmax > 0
    assert (gmax[nz] <= 7 * np.exp2(e[nz].astype(np.float64))).all() and (gmax[nz] > 7 * np.exp2(e[nz].astype(np.float64) - 1)).all()
    assert (e[~nz] == -126).all() and (d[3, 64:128] == 0).all()
    # dequantised weights are bf16 values, and quantising them again changes nothing
    assert torch.equal(torch.from_numpy(d).to(torch.bfloat16).float(), torch.from_numpy(d))
    q2, e2 = orc.quantize_int4(d)
    d2 = orc.dequantize_int4(q2, e2)
    assert np.array_equal(d2, d)
    # a linear layer over the quantised weights is the plain linear layer over the dequantised ones
    x = rng.standard_normal((3, 256))
    assert np.allclose(orc.linear(d, x), x @ d.astype(np.float64).T, rtol=1e-12, atol=1e-12)
