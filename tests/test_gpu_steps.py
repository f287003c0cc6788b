"""GPU parity of the single steps (mask table, search + rollback, skinny GEMM, tree attention)
against the CPU oracle, through the C ABI."""
import os

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2309_04255_b200 import binding as B
from paper_2309_04255_b200 import inputs as gen

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
DEV = "cuda:0"


def dev_i32(a):
    return torch.as_tensor(np.asarray(a, np.int32), device=DEV)


def trees():
    yield np.array([-1], np.int32)
    yield np.array([-1, 0, 1, 2, 2, 3, 4], np.int32)          # the paper's mask example
    yield gen.tree_chain(128)
    yield gen.tree_star(128)
    yield gen.tree_binary(4)
    yield gen.tree_binary(7)
    for s in range(6):
        yield gen.tree_random(8 + 24 * s, 4 + 2 * s, "uniform4" if s % 2 else "geometric4", s)


# ----------------------------------------------------------------------------- mask table

@pytest.mark.parametrize("idx", range(12))
def test_tree_prep_bit_exact(idx):
    parent = list(trees())[idx]
    n = len(parent)
    for P in (0, 517):
        depth, pos, anc, status = B.tree_prep(dev_i32(parent), P)
        st, odepth, opos, oanc = orc.tree_prep(parent, P)
        assert st == 0 and int(status.item()) == 0
        assert (depth.cpu().numpy() == odepth).all()
        assert (pos.cpu().numpy() == opos).all()
        assert (B.anc_to_bool(anc.cpu().numpy(), n) == oanc).all()


@pytest.mark.parametrize("bad", [[0, 0, 1], [-1, -1, 0], [-1, 1, 0], [-1, 0, 3], [-1, 5], [-2, 0]])
def test_tree_prep_rejects_bad_trees(bad):
    *_, status = B.tree_prep(dev_i32(bad), 3)
    assert int(status.item()) == B.ERR_BAD_TREE
    assert orc.tree_prep(bad, 3)[0] == 1


# ----------------------------------------------------------------------------- search + rollback

def small_cfg(dtype="bf16", L=3, H=2, hd=128):
    return gen.ModelConfig("small", L, H * hd, H, hd, 256, 512, dtype)


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                k, v = line.split(":")
                out[k.strip()] = [int(t) for t in v.split()]
    return out


def test_accept_paper_example():
    g = read_golden("acceptance_example.txt")
    cfg = gen.ModelConfig("small", 1, 256, 2, 128, 256, 1024, "bf16")
    v = B.Verifier(cfg, 64)
    path, sc = v.accept_compact(5, dev_i32(g["tokens"]), dev_i32(g["parent_idx"]), dev_i32(g["argmax"]), compact=False)
    sc = sc.cpu().numpy()
    assert sc[B.S_STATUS] == 0
    assert path.cpu().numpy()[: sc[B.S_ACCEPTED_LEN]].tolist() == g["path"]
    assert sc[B.S_NEXT_TOKEN] == g["next_token"][0] and sc[B.S_RECTIFIED] == g["rectified"][0]
    assert sc[B.S_NEW_PREFIX_LEN] == 5 + len(g["path"])


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("seed", range(8))
def test_accept_compact_random(seed, dtype):
    """Small vocabulary: many matches, duplicate sibling tokens. The path and scalars equal the
    oracle's depth-first search; the cache equals 'prefix rows, then the path's rows' bit for bit."""
    g = np.random.default_rng(seed)
    cfg = small_cfg(dtype)
    n = [1, 2, 17, 40, 77, 128, 128, 100][seed]
    P = [0, 3, 11, 64, 100, 7, 0, 33][seed]
    parent = gen.tree_chain(n) if seed == 5 else (gen.tree_random(n, 12, "uniform4", seed) if n > 1 else np.array([-1], np.int32))
    V = 2 if seed != 5 else 1      # seed 5: chain with every token accepted -> all 128 rows move
    tokens = g.integers(0, V, n).astype(np.int32)
    amax = g.integers(0, V, n).astype(np.int32)
    v = B.Verifier(cfg, P + n + 5)
    kvv = v.kv_view()
    kvv.copy_(torch.randn(kvv.shape, device=DEV).to(kvv.dtype))
    before = kvv.clone()
    path, sc = v.accept_compact(P, dev_i32(tokens), dev_i32(parent), dev_i32(amax))
    torch.cuda.synchronize()
    sc = sc.cpu().numpy()
    acc = orc.accept(parent, tokens, amax)
    assert sc[B.S_STATUS] == 0
    assert sc[B.S_ACCEPTED_LEN] == acc.accepted_len and sc[B.S_NEXT_TOKEN] == acc.next_token
    assert sc[B.S_N_CORRECT] == acc.n_correct and sc[B.S_N_ALL] == acc.n_all and sc[B.S_RECTIFIED] == acc.rectified
    assert sc[B.S_NEW_PREFIX_LEN] == P + acc.accepted_len
    assert path.cpu().numpy()[: acc.accepted_len].tolist() == acc.path.tolist()
    after = v.kv_view()
    assert torch.equal(after[:, :, :, :P], before[:, :, :, :P])          # prefix untouched
    idx = torch.as_tensor(P + acc.path.astype(np.int64), device=DEV)
    assert torch.equal(after[:, :, :, P:P + acc.accepted_len], before[:, :, :, idx])


def test_accept_reports_bad_tree_and_leaves_cache():
    cfg = small_cfg()
    v = B.Verifier(cfg, 64)
    kvv = v.kv_view()
    kvv.copy_(torch.randn(kvv.shape, device=DEV).to(kvv.dtype))
    before = kvv.clone()
    path, sc = v.accept_compact(4, dev_i32([1, 1, 1]), dev_i32([-1, 2, 0]), dev_i32([1, 1, 1]))
    sc = sc.cpu().numpy()
    assert sc[B.S_STATUS] == B.ERR_BAD_TREE and sc[B.S_ACCEPTED_LEN] == 0 and sc[B.S_NEW_PREFIX_LEN] == 4
    assert torch.equal(v.kv_view(), before)


# ----------------------------------------------------------------------------- skinny GEMM

GEMM_SHAPES = [
    # n_out, n_in, n: several 128-row tiles with a ragged last tile, k-ranges split over CTAs
    (300, 256, 15), (128, 64, 1), (688, 256, 15), (1024, 688, 33), (4096, 4096, 32), (4096, 11008, 32),
    (1000, 2048, 128), (12288, 4096, 64), (2500, 520, 17),
]


@pytest.mark.parametrize("shape", GEMM_SHAPES)
@pytest.mark.parametrize("mode", ["f32", "bf16_simt", "bf16_tc", "bf16_tc_tiled"])
def test_skinny_gemm(shape, mode):
    n_out, n_in, n = shape
    g = np.random.default_rng(n_out + n_in + n)
    dtype = "f32" if mode == "f32" else "bf16"
    cfg = gen.ModelConfig("g", 0, 256, 2, 128, 256, 512, dtype)
    v = B.Verifier(cfg, 16, flags=B.FLAG_SIMT_GEMM if mode == "bf16_simt" else 0)
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    W = torch.from_numpy(g.standard_normal((n_out, n_in), dtype=np.float32)).to(td)
    x = torch.from_numpy(g.standard_normal((n, n_in), dtype=np.float32)).to(td)
    if mode == "bf16_tc_tiled":     # the layout the pass itself streams (pre-swizzled 16 KB tiles)
        y = v.skinny_gemm_tiled(v.tile_weight(W.to(DEV)), n_out, x.to(DEV))
    else:
        y = v.skinny_gemm(W.to(DEV), x.to(DEV))
    assert v.last_status() == 0
    ref = orc.linear(W, x.double())
    # inputs are identical on both sides and products are exact in fp32; only the order of the
    # fp32 accumulation differs: error ~ sqrt(n_in) * 2^-24 * |terms|
    scale = np.abs(ref).max()
    err = np.abs(y.cpu().numpy() - ref).max()
    assert err <= 2e-5 * scale, (err, scale)


# ----------------------------------------------------------------------------- tree attention

ATTN_CASES = [(0, 1), (0, 15), (5, 8), (64, 33), (300, 32), (1024, 64), (257, 128), (2048, 17), (1000, 97), (4095, 128),
              # fewer query rows than key splits (some CTAs of a cluster own no row), uneven tiles per split
              (2048, 1), (500, 3), (129, 16), (577, 32)]


@pytest.mark.parametrize("case", ATTN_CASES)
@pytest.mark.parametrize("mode", ["f32", "bf16_simt", "bf16_mma", "bf16_t5"])
def test_tree_attention(case, mode):
    """Every attention kernel family on every shape: plain ALU (fp32, bf16), mma.sync and tcgen05."""
    P, n = case
    H, hd = 4, 128
    dtype = "f32" if mode == "f32" else "bf16"
    cfg = gen.ModelConfig("a", 0, H * hd, H, hd, 256, 512, dtype)
    flags = {"f32": 0, "bf16_simt": B.FLAG_SIMT_ATTN, "bf16_mma": B.FLAG_MMA_ATTN, "bf16_t5": B.FLAG_T5_ATTN}[mode]
    v = B.Verifier(cfg, 16, flags=flags)
    if n == 1:
        parent = np.array([-1], np.int32)
    elif n == 15:
        parent = gen.tree_binary(4)
    else:
        parent = gen.tree_random(n, 12, "uniform4", P + n)
    q, k, vv = gen.gen_attention_inputs(H, hd, P, n, seed=1, dtype=dtype)
    stride = P + n + 3                       # rows past the end hold NaN: they must never be read into a result
    kbuf = torch.full((H, stride, hd), float("nan"), dtype=q.dtype)
    vbuf = torch.full((H, stride, hd), float("nan"), dtype=q.dtype)
    kbuf[:, :P + n] = k
    vbuf[:, :P + n] = vv
    o = v.tree_attention(q.to(DEV), kbuf.to(DEV), vbuf.to(DEV), P, dev_i32(parent))
    assert v.last_status() == 0
    _, _, _, anc = orc.tree_prep(parent, P)
    tk = k[:, P:].permute(1, 0, 2).reshape(n, H * hd)
    tv = vv[:, P:].permute(1, 0, 2).reshape(n, H * hd)
    ref = orc.tree_attention(q.reshape(n, H * hd), k[:, :P], vv[:, :P], tk, tv, anc, H, hd)
    got = o.double().cpu().numpy().reshape(n, H * hd)
    assert np.isfinite(got).all()
    tol = 1e-5 if dtype == "f32" else 2e-2
    assert np.abs(got - ref).max() <= tol * np.abs(ref).max()


# Config 4 at its own head count and its extreme prefix lengths: with 32 heads there are fewer key
# splits per head than in the 4-head cases above, so the cluster and merge shapes differ.
C4_CASES = [(P, n, "random") for P in (256, 8192) for n in (8, 32, 64, 128)] + [(8192, 128, "chain"), (8192, 128, "star")]


@pytest.mark.parametrize("case", C4_CASES)
@pytest.mark.parametrize("mode", ["bf16_mma", "bf16_t5"])
def test_tree_attention_config4(case, mode):
    """32 heads x 128, prefix 256 and 8192, trees of 8..128 nodes (random, chain, star), each tensor
    kernel pinned, element by element against the oracle."""
    P, n, shape = case
    H, hd = 32, 128
    cfg = gen.ModelConfig("a", 0, H * hd, H, hd, 256, 512, "bf16")
    v = B.Verifier(cfg, 16, flags={"bf16_mma": B.FLAG_MMA_ATTN, "bf16_t5": B.FLAG_T5_ATTN}[mode])
    parent = {"random": lambda: gen.tree_random(n, 12, "uniform4", P + n), "chain": lambda: gen.tree_chain(n),
              "star": lambda: gen.tree_star(n)}[shape]()
    q, k, vv = gen.gen_attention_inputs(H, hd, P, n, seed=2, dtype="bf16")
    o = v.tree_attention(q.to(DEV), k.to(DEV), vv.to(DEV), P, dev_i32(parent))
    assert v.last_status() == 0
    _, _, _, anc = orc.tree_prep(parent, P)
    tk = k[:, P:].permute(1, 0, 2).reshape(n, H * hd)
    tv = vv[:, P:].permute(1, 0, 2).reshape(n, H * hd)
    ref = orc.tree_attention(q.reshape(n, H * hd), k[:, :P], vv[:, :P], tk, tv, anc, H, hd)
    got = o.double().cpu().numpy().reshape(n, H * hd)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= 2e-2 * np.abs(ref).max()


@pytest.mark.parametrize("mode", ["bf16_mma", "bf16_t5"])
def test_tree_attention_refuses_a_malformed_tree_of_40_nodes(mode):
    """Above 32 nodes the default kernel is the tcgen05 one: it too must leave o alone and report the tree."""
    P, n, H, hd = 70, 40, 4, 128
    cfg = gen.ModelConfig("a", 0, H * hd, H, hd, 256, 512, "bf16")
    v = B.Verifier(cfg, 16, flags={"bf16_mma": B.FLAG_MMA_ATTN, "bf16_t5": B.FLAG_T5_ATTN}[mode])
    parent = gen.tree_random(n, 12, "uniform4", 5)
    parent[35] = 37                                    # a parent that comes after its child
    q, k, vv = gen.gen_attention_inputs(H, hd, P, n, seed=4, dtype="bf16")
    o = torch.full((n, H, hd), 7.0, dtype=torch.bfloat16, device=DEV)
    v.tree_attention(q.to(DEV), k.to(DEV), vv.to(DEV), P, dev_i32(parent), o=o)
    assert v.last_status() == B.ERR_BAD_TREE
    assert (o == 7.0).all()                            # nothing was written
    # a well-formed call afterwards works and differs from what the refused call left behind
    parent[35] = 3
    o2 = v.tree_attention(q.to(DEV), k.to(DEV), vv.to(DEV), P, dev_i32(parent))
    assert v.last_status() == 0 and torch.isfinite(o2.float()).all()
    # misaligned buffers are refused on the host
    qd = torch.zeros(n * H * hd + 8, dtype=torch.bfloat16, device=DEV)[4:4 + n * H * hd].view(n, H, hd)
    with pytest.raises(B.LlmcadError) as e:
        v.tree_attention(qd, k.to(DEV), vv.to(DEV), P, dev_i32(parent))
    assert e.value.code == B.ERR_INVALID_ARG


def test_attention_head_dim_64_f32():
    P, n, H, hd = 40, 15, 4, 64
    cfg = gen.ModelConfig("a", 0, H * hd, H, hd, 256, 512, "f32")
    v = B.Verifier(cfg, 16)
    parent = gen.tree_binary(4)
    q, k, vv = gen.gen_attention_inputs(H, hd, P, n, seed=2, dtype="f32")
    o = v.tree_attention(q.to(DEV), k.to(DEV), vv.to(DEV), P, dev_i32(parent))
    _, _, _, anc = orc.tree_prep(parent, P)
    ref = orc.tree_attention(q.reshape(n, H * hd), k[:, :P], vv[:, :P], k[:, P:].permute(1, 0, 2).reshape(n, -1),
                             vv[:, P:].permute(1, 0, 2).reshape(n, -1), anc, H, hd)
    assert np.abs(o.double().cpu().numpy().reshape(n, -1) - ref).max() <= 1e-5 * np.abs(ref).max()


# ----------------------------------------------------------------------------- machine probes (measurement interface)

def test_machine_probes_run_and_are_plausible():
    """The micro-benchmarks of llmcad_profile.h return sane figures: a streaming read well above 1 TB/s with a
    latency of microseconds at most, and an mma.sync rate between 100 and 4096 multiply-adds per clock and SM."""
    src = torch.ones(1 << 30, dtype=torch.uint8, device=DEV)
    gbs, lat = B.probe_bulk_copy(src, 32768, 4)
    assert 1000.0 < gbs < 20000.0 and 0.1 < lat < 50.0, (gbs, lat)
    gbs1, _ = B.probe_bulk_copy(src, 8448, 1)
    assert gbs1 < gbs
    rate, cyc = B.probe_mma_sync(8, 8)
    assert 100.0 < rate <= 4096.0 and cyc > 1.0, (rate, cyc)
    with pytest.raises(B.LlmcadError):
        B.probe_bulk_copy(src, 1000, 4)          # not a multiple of 16
