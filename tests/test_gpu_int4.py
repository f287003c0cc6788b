"""INT4 weights (Sec. 4.1): the quantisation kernel against the oracle's codes bit for bit, the
streaming GEMM over INT4 tiles against the oracle's linear layer over the dequantised weights, and
whole passes of an INT4 context against (a) the oracle pass over the dequantised weights and (b) a
bf16 context that was handed the dequantised weights: (b) must agree bit for bit, because every
dequantised weight is a bf16 value and the kernel expands the codes to exactly those tiles."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2309_04255_b200 import binding as B
from paper_2309_04255_b200 import inputs as gen

from gpu_util import BF16_TOL, Twin, argmax_agrees_where_decided, check_acceptance_against_oracle, logits_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("shape", [(300, 256), (128, 64), (1000, 2048), (4096, 11008)])
def test_quantisation_codes_are_the_oracles(shape):
    n_out, n_in = shape
    g = np.random.default_rng(n_out + n_in)
    w = torch.from_numpy((g.standard_normal((n_out, n_in)) * 0.02).astype(np.float32)).to(torch.bfloat16)
    w[1, :64] = 0                       # a group of zeros
    w[2, 5] = 3.0                       # an outlier
    w[3, :64] = w[3, :64].abs().max()   # plateau: every element at the group maximum
    w[4, :64] = 0.875                    # the maximum exactly on a scale boundary (7 * 2^-3)
    q, e = B.quantize_int4(w.to(DEV))
    q_ref, e_ref = orc.quantize_int4(w)
    assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(e.cpu().numpy(), e_ref)


GEMM_SHAPES = [(300, 256, 15), (128, 64, 1), (1024, 704, 33), (4096, 4096, 32), (4096, 11008, 32), (1000, 2048, 128), (12288, 4096, 64)]


@pytest.mark.parametrize("shape", GEMM_SHAPES)
def test_skinny_gemm_over_int4_tiles(shape):
    n_out, n_in, n = shape
    g = np.random.default_rng(n_out + n_in + n)
    cfg = gen.ModelConfig("g", 0, 256, 2, 128, 256, 512, "bf16")
    v = B.Verifier(cfg, 16)
    W = torch.from_numpy((g.standard_normal((n_out, n_in)) * 0.02).astype(np.float32)).to(torch.bfloat16)
    x = torch.from_numpy(g.standard_normal((n, n_in), dtype=np.float32)).to(torch.bfloat16)
    y = v.skinny_gemm_tiled_int4(v.tile_weight_int4(W.to(DEV)), n_out, x.to(DEV))
    assert v.last_status() == 0
    Wd = orc.dequantize_int4(*orc.quantize_int4(W))
    ref = orc.linear(Wd, x.double())
    scale = np.abs(ref).max()
    # identical inputs on both sides, exact products: only the order of the fp32 accumulation differs
    assert np.abs(y.cpu().numpy() - ref).max() <= 2e-5 * scale
    # and the same GEMM over the dequantised weights as bf16 tiles gives the same bits
    y2 = v.skinny_gemm_tiled(v.tile_weight(torch.from_numpy(Wd).to(torch.bfloat16).to(DEV)), n_out, x.to(DEV))
    assert torch.equal(y, y2)


class Int4Twin(Twin):
    """An INT4 context next to a bf16 context that holds the dequantised weights; the oracle uses those too."""

    def __init__(self, cfg, max_seq, scale=1.0, seed=0):
        super().__init__(cfg, max_seq, flags=B.FLAG_INT4_WEIGHTS, seed=seed, scale=scale)
        self.v16 = B.Verifier(cfg, max_seq)
        self.v16.pack_globals(self.glob)
        self.dq = {}
        for l in range(cfg.n_layers):
            self.dq[l] = {k: (torch.from_numpy(t).to(torch.bfloat16) if isinstance(t, np.ndarray) else t)
                          for k, t in orc.int4_weights(self.layers[l]).items()}
            self.v16.pack_layer(l, self.dq[l])

    def layer(self, l):
        return self.dq[l]


@pytest.mark.parametrize("case", [("small", 2, 100, 20), ("small", 2, 64, 128), ("7b", 2, 300, 32), ("13b", 1, 200, 64)])
def test_int4_pass_against_oracle_and_against_bf16_over_dequantised_weights(case):
    name, layers, P, n = case
    cfg = gen.ModelConfig("small-bf16", 2, 512, 4, 128, 1408, 2048, "bf16") if name == "small" else gen.shrink(gen.MODELS[name], layers)
    twin = Int4Twin(cfg, P + n + 8, scale=3.0 if name == "small" else 1.0, seed=n)
    twin.fill_prefix_synthetic(P)
    kv16 = twin.v16.kv_view()
    kv16[:, :, :, :P] = twin.v.kv_view()[:, :, :, :P]
    parent = gen.tree_random(n, 10, "uniform4", n)
    tokens = gen.gen_tokens(cfg, n, seed=n)
    out = twin.gpu_pass(P, tokens, parent)
    for it in range(3):                      # plant the device's own argmax so that a real path gets verified
        tokens = gen.plant_tokens(parent, tokens, out["argmax"], seed=it, prob=0.9)
        out = twin.gpu_pass(P, tokens, parent)
    ref = twin.oracle_pass(P, tokens, parent)
    logits_close(out["logits"], ref.logits, BF16_TOL)
    logits_close(out["logits"], ref.logits, 1e-3)
    argmax_agrees_where_decided(out["argmax"], ref.logits, BF16_TOL)
    check_acceptance_against_oracle(out, tokens, parent)
    # the bf16 context over the dequantised weights: same bits everywhere
    t = torch.as_tensor(np.asarray(tokens, np.int32), device=DEV)
    p = torch.as_tensor(np.asarray(parent, np.int32), device=DEV)
    o16 = twin.v16.verify_tree(P, t, p)
    torch.cuda.synchronize()
    assert np.array_equal(o16["logits"].cpu().numpy(), out["logits"])
    assert np.array_equal(o16["scalars"].cpu().numpy(), out["scalars"])
    L = int(out["scalars"][B.S_ACCEPTED_LEN])
    assert torch.equal(twin.v16.kv_view()[:, :, :, :P + L], twin.v.kv_view()[:, :, :, :P + L])
    # a quarter of the weight bytes (plus the exponents)
    c4, c16 = B.make_config(cfg, 64, flags=B.FLAG_INT4_WEIGHTS), B.make_config(cfg, 64)
    import ctypes
    layer_bytes = lambda c: B.lib().llmcad_packed_weight_bytes(ctypes.byref(c)) - 2 * cfg.vocab * cfg.d_model * 2
    assert layer_bytes(c4) < 0.27 * layer_bytes(c16)


def test_int4_contexts_are_refused_where_they_cannot_work():
    import ctypes
    h = ctypes.c_void_p()
    c = B.make_config(gen.MODELS["tiny"], 64, flags=B.FLAG_INT4_WEIGHTS)         # fp32
    assert B.lib().llmcad_create(ctypes.byref(c), ctypes.byref(h)) == B.ERR_UNSUPPORTED
    cfg = gen.ModelConfig("odd", 1, 512, 4, 128, 1000, 512, "bf16")               # FFN width not a multiple of 64
    c = B.make_config(cfg, 64, flags=B.FLAG_INT4_WEIGHTS)
    assert B.lib().llmcad_create(ctypes.byref(c), ctypes.byref(h)) == B.ERR_UNSUPPORTED


def test_int4_passes_of_changing_prefix_and_size_are_reproducible():
    """Passes over different prefix lengths and tree sizes, queued back to back on one INT4 context, each give bit
    for bit what the same pass gave the first time (the cache is put back before every pass, since a pass writes
    its tree nodes' slots): the three rings of the INT4 GEMMs and the split merge of the attention kernels leave
    nothing behind that depends on timing or on the previous launch's shape."""
    cfg = gen.shrink(gen.MODELS["7b"], 2)
    S = 640 + 136
    v = B.Verifier(cfg, S, device=DEV, flags=B.FLAG_INT4_WEIGHTS)
    v.pack_globals({k: gen.gen_tensor_device(cfg, k, -1, DEV) for k in ("tok_embed", "final_norm", "lm_head")})
    for l in range(cfg.n_layers):
        v.pack_layer(l, {k: gen.gen_tensor_device(cfg, k, l, DEV) for k in gen.LAYER_TENSORS})
    kvv = v.kv_view()
    kvv[:, :, :, :640] = torch.randn((cfg.n_layers, 2, cfg.n_heads, 640, cfg.head_dim), device=DEV).to(kvv.dtype)
    saved = kvv.clone()
    cases = []
    for P in (1, 64, 577, 640):
        for n in (1, 17, 32, 33, 128):
            tokens = torch.as_tensor(gen.gen_tokens(cfg, n, seed=n + P), device=DEV)
            parent = torch.as_tensor(gen.tree_random(n, 12, "uniform4", n + P) if n > 1 else np.array([-1], np.int32), device=DEV)
            kvv.copy_(saved)
            out = v.verify_tree(P, tokens, parent)
            torch.cuda.synchronize()
            assert out["scalars"][B.S_STATUS].item() == 0
            cases.append((P, n, tokens, parent, out["logits"].clone(), out["scalars"].clone()))
    rng = np.random.default_rng(3)
    outs = []
    for _ in range(200):
        ci = int(rng.integers(len(cases)))
        P, n, tokens, parent, _, _ = cases[ci]
        kvv.copy_(saved)
        o = v.new_outputs(n)
        v.verify_tree(P, tokens, parent, out=o)
        outs.append((ci, o))
    torch.cuda.synchronize()
    for ci, o in outs:
        assert torch.equal(o["logits"], cases[ci][4]) and torch.equal(o["scalars"], cases[ci][5]), cases[ci][:2]
    v.close()
