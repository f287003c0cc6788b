"""The allocation-free tree-attention entry point against the regular one.

llmcad_tree_attention_noalloc serves callers that must not allocate device memory (a plug-in
inside a server whose pool already owns the device, a loop where cudaMalloc's device-wide
synchronisation is not acceptable): it takes no context and keeps its scratch in a static device
array. Here it is called twice in a row through the C ABI, on different trees, and each result
must equal what llmcad_tree_attention gives for the same inputs (same kernels, same arithmetic:
bit-identical, which is within the 2e-2 tolerance the other bf16 tests use). The file sorts last
so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2309_04255_b200 import binding as B
from paper_2309_04255_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def test_noalloc_matches_regular_entry_point_twice():
    dev = torch.device("cuda:0")
    H, hd = 8, 128
    cfg = gen.ModelConfig("a", 0, H * hd, H, hd, 256, 512, "bf16")
    ref = B.Verifier(cfg, 16)                    # the regular entry point needs a context
    cases = [(300, 24, 1), (77, 128, 2)]         # (prefix, nodes, seed): the second reuses the scratch of the first
    for P, n, seed in cases:
        parent = torch.as_tensor(gen.tree_random(n, 12, "uniform4", seed), device=dev)
        q, k, v = (t.to(dev) for t in gen.gen_attention_inputs(H, hd, P, n, seed=seed))
        want = ref.tree_attention(q, k, v, P, parent)
        got = torch.full_like(q, float("nan"))
        status = torch.full((1,), -7, dtype=torch.int32, device=dev)
        if seed == 1:
            # the very first call loads the kernels' module and looks up the scratch address; what
            # must not allocate is every call, so the free-memory reading brackets a call after it
            B.tree_attention_noalloc(q, k, v, P, parent, got, status)
            torch.cuda.synchronize()
            got.fill_(float("nan"))
        # free device memory as the driver reports it (cudaMemGetInfo): an allocation by the
        # library itself, which torch's own counters cannot see, would lower it
        free_before, _ = torch.cuda.mem_get_info(dev)
        B.tree_attention_noalloc(q, k, v, P, parent, got, status)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info(dev)
        assert free_after == free_before
        assert int(status.item()) == 0
        g, w = got.float().cpu().numpy(), want.float().cpu().numpy()
        assert np.isfinite(g).all()
        assert np.abs(g - w).max() <= 2e-2 * np.abs(w).max()
        assert np.array_equal(g, w)              # same kernels on the same inputs
        # and directly against the CPU oracle's tree attention
        par = parent.cpu().numpy()
        _, _, _, anc = orc.tree_prep(par, P)
        kc, vc = k.cpu(), v.cpu()
        ref_o = orc.tree_attention(q.cpu().reshape(n, H * hd), kc[:, :P], vc[:, :P], kc[:, P:].permute(1, 0, 2).reshape(n, H * hd),
                                   vc[:, P:].permute(1, 0, 2).reshape(n, H * hd), anc, H, hd)
        assert np.abs(got.double().cpu().numpy().reshape(n, H * hd) - ref_o).max() <= 2e-2 * np.abs(ref_o).max()
    # a malformed tree is reported through the status word, which the previous calls left at 0
    bad = torch.as_tensor(np.array([-1, 2, 0], np.int32), device=dev)
    q, k, v = (t.to(dev) for t in gen.gen_attention_inputs(H, hd, 5, 3, seed=3))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.tree_attention_noalloc(q, k, v, 5, bad, torch.empty_like(q), status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.ERR_BAD_TREE
    # and the call after that starts from a clean status again
    good = torch.as_tensor(np.array([-1, 0, 0], np.int32), device=dev)
    B.tree_attention_noalloc(q, k, v, 5, good, torch.empty_like(q), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # the same with a tree large enough for the tcgen05 kernel: refused, and o left as it was
    n = 40
    par = gen.tree_random(n, 12, "uniform4", 9)
    par[30] = 33
    q, k, v = (t.to(dev) for t in gen.gen_attention_inputs(H, hd, 20, n, seed=5))
    o = torch.full_like(q, 7.0)
    B.tree_attention_noalloc(q, k, v, 20, torch.as_tensor(par, device=dev), o, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.ERR_BAD_TREE and bool((o == 7.0).all())
    # buffers the kernels could not read as 16-byte vectors are refused before anything is launched
    flat = torch.zeros(q.numel() + 8, dtype=torch.bfloat16, device=dev)
    with pytest.raises(B.LlmcadError) as e:
        B.tree_attention_noalloc(flat[4:4 + q.numel()].view(q.shape), k, v, 20, torch.as_tensor(par, device=dev), o, status)
    assert e.value.code == B.ERR_INVALID_ARG


def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    dev = torch.device("cuda:0")
    H, hd, n = 2, 128, 129
    q = torch.zeros((n, H, hd), dtype=torch.bfloat16, device=dev)
    k = torch.zeros((H, n + 4, hd), dtype=torch.bfloat16, device=dev)
    parent = torch.zeros(n, dtype=torch.int32, device=dev)
    with pytest.raises(B.LlmcadError) as e:
        B.tree_attention_noalloc(q, k, k, 4, parent, torch.empty_like(q))
    assert e.value.code == B.ERR_UNSUPPORTED and "128" in str(e.value)
