"""Tree extension (the tree decoder on the generating side): a tree grown in several calls of
llmcad_extend_tree must give, for every node, the logits that one pass over the finished tree
gives (the oracle's pass is the definition; it has no incremental form), and the top-k
confidences must be the softmax of those logits."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2309_04255_b200 import binding as B
from paper_2309_04255_b200 import inputs as gen

from gpu_util import BF16_TOL, F32_TOL, Twin, logits_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def grow(twin, P, tokens, parent, cuts, k):
    """Extends the tree in the steps given by `cuts` (node counts after each call); returns the
    concatenated logits, ids and probabilities of all nodes."""
    lg, ids, pr = [], [], []
    n_old = 0
    for n_tree in cuts:
        out = twin.v.extend_tree(P, torch.as_tensor(tokens[:n_tree], device=DEV), torch.as_tensor(parent[:n_tree], device=DEV),
                                 n_old, top_k=k)
        torch.cuda.synchronize()
        assert out["status"].item() == 0
        lg.append(out["logits"].cpu().numpy()); ids.append(out["topk_ids"].cpu().numpy()); pr.append(out["topk_probs"].cpu().numpy())
        n_old = n_tree
    return np.concatenate(lg), np.concatenate(ids), np.concatenate(pr)


def check_topk(ids, probs, ref_logits, tol_scale):
    """ids: where the oracle's k-th and (k+1)-th logits are further apart than the tolerance the
    sets must agree; probabilities against the oracle's softmax of its own logits."""
    k = ids.shape[1]
    rid, rpr = orc.topk_softmax(ref_logits, k + 1)
    srt = -np.sort(-ref_logits, axis=1)
    for i in range(ids.shape[0]):
        gaps = srt[i, :k] - srt[i, 1:k + 1]
        if gaps.min() > tol_scale:
            assert ids[i].tolist() == rid[i, :k].tolist()
            np.testing.assert_allclose(probs[i], rpr[i, :k], rtol=0, atol=4 * tol_scale * rpr[i, :k].max() + 1e-7)
    assert np.all(np.diff(probs, axis=1) <= 1e-7)


def test_extension_fp32_tiny_tree_in_four_steps():
    w = gen.WORKLOADS["C1"]
    cfg = gen.MODELS[w.model]
    tw = Twin(cfg, w.prefix_len + w.n_nodes + 8)
    P = w.prefix_len
    tw.fill_prefix_synthetic(P)
    parent = gen.gen_tree(w)
    tokens = gen.gen_tokens(cfg, w.n_nodes)
    ref = tw.oracle_pass(P, tokens, parent)
    lg, ids, pr = grow(tw, P, tokens, parent, [1, 5, 9, w.n_nodes], 4)
    logits_close(lg, ref.logits, F32_TOL)
    check_topk(ids, pr, ref.logits, F32_TOL * np.abs(ref.logits).max())
    # and the finished tree verified in one pass gives the same logits as the extensions did
    out = tw.v.verify_tree(P, torch.as_tensor(tokens, device=DEV), torch.as_tensor(parent, device=DEV))
    torch.cuda.synchronize()
    logits_close(out["logits"].cpu().numpy(), lg.astype(np.float64), F32_TOL)


@pytest.mark.parametrize("cuts", [[32], [16, 32], [3, 4, 20, 31, 32]])
def test_extension_bf16_full_width(cuts):
    """7B widths, two layers, 32 nodes: whole tree at once (n_old = 0) and in uneven steps. Nodes added
    earlier are read back from the cache rounded to bf16, like the prefix."""
    w = gen.WORKLOADS["C2"]
    cfg = gen.shrink(gen.MODELS[w.model], 2)
    tw = Twin(cfg, w.prefix_len + w.n_nodes + 8)
    P = w.prefix_len
    tw.fill_prefix_synthetic(P)
    parent = gen.gen_tree(w)
    tokens = gen.gen_tokens(cfg, w.n_nodes)
    ref = tw.oracle_pass(P, tokens, parent)
    lg, ids, pr = grow(tw, P, tokens, parent, cuts, 8)
    logits_close(lg, ref.logits, BF16_TOL)
    check_topk(ids, pr, ref.logits, BF16_TOL * np.abs(ref.logits).max())


@pytest.mark.parametrize("flags,n,cuts", [(B.FLAG_T5_ATTN, 32, [3, 4, 20, 31, 32]), (B.FLAG_MMA_ATTN, 32, [3, 4, 20, 31, 32]),
                                          (0, 96, [40, 41, 96])])
def test_extension_through_both_attention_kernels(flags, n, cuts):
    """The same at 7B widths with each tensor-core attention kernel pinned (a query block that starts
    inside the tree, remainders only for the new nodes), and a 96-node tree grown by 40, 1 and 55 nodes,
    which the default choice sends to the tcgen05, the mma.sync and again the tcgen05 kernel."""
    cfg = gen.shrink(gen.MODELS["7b"], 2)
    P = 300
    tw = Twin(cfg, P + n + 8, flags=flags)
    tw.fill_prefix_synthetic(P)
    parent = gen.tree_random(n, 12, "uniform4", n)
    tokens = gen.gen_tokens(cfg, n)
    ref = tw.oracle_pass(P, tokens, parent)
    lg, ids, pr = grow(tw, P, tokens, parent, cuts, 4)
    logits_close(lg, ref.logits, BF16_TOL)
    check_topk(ids, pr, ref.logits, BF16_TOL * np.abs(ref.logits).max())


def test_extension_argument_checks():
    cfg = gen.MODELS["tiny"]
    v = B.Verifier(cfg, 64)
    t = torch.zeros(4, dtype=torch.int32, device=DEV)
    p = torch.as_tensor(np.array([-1, 0, 1, 2], np.int32), device=DEV)
    with pytest.raises(B.LlmcadError):
        v.extend_tree(8, t, p, 4)            # nothing new
    with pytest.raises(B.LlmcadError):
        v.extend_tree(8, t, p, 0, top_k=9)   # more than LLMCAD_MAX_TOPK
    with pytest.raises(B.LlmcadError):
        v.extend_tree(62, t, p, 0)           # beyond the cache
