"""Seeded synthetic inputs for token-tree verification.

This module serves both the CUDA path and the CPU oracle with the same bytes.
It holds generators only (model shapes, random weights, random prefix K/V,
random draft trees and their tokens); none of the method's arithmetic lives
here.

The paper evaluates on public text datasets with trained checkpoints; none of
that is available offline, so every input is synthetic:

* weights ~ N(0, 0.02), one independent stream per (layer, tensor, block of 1024
  rows), rounded to bf16 for the bf16 configurations; RMSNorm gains are 1.0;
* prefix K/V ~ N(0, 1) (the natural scale of q = x_hat W with std 0.02 sqrt(d));
* draft trees follow the paper's draft rule (a successor opens a branch when its
  confidence exceeds ~30 %, hence at most 3-4 children per node; branches are
  2-10 tokens long; up to tens of branches).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional

import numpy as np
import torch

MASTER_SEED = 20230904

# tensor ids used in the per-tensor seed derivation
_TID = {
    "tok_embed": 1, "final_norm": 2, "lm_head": 3,
    "attn_norm": 10, "wq": 11, "wk": 12, "wv": 13, "wo": 14,
    "ffn_norm": 15, "w_gate": 16, "w_up": 17, "w_down": 18,
    "prefix_k": 30, "prefix_v": 31, "q": 32,
}
LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


@dataclass(frozen=True)
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: str  # "f32" or "bf16"
    rms_eps: float = 1e-5
    rope_base: float = 10000.0

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def layer_weight_elems(self) -> int:
        d, f = self.d_model, self.d_ffn
        return 4 * d * d + 3 * d * f

    def weight_bytes(self) -> int:
        """Bytes one pass must read: every layer matrix once plus the lm_head."""
        return (self.n_layers * self.layer_weight_elems() + self.vocab * self.d_model) * self.elem_bytes


MODELS: Dict[str, ModelConfig] = {
    "tiny": ModelConfig("tiny", 2, 256, 4, 64, 688, 1024, "f32"),
    "7b": ModelConfig("7b", 32, 4096, 32, 128, 11008, 32000, "bf16"),
    "13b": ModelConfig("13b", 40, 5120, 40, 128, 13824, 32000, "bf16"),
    "30b": ModelConfig("30b", 60, 6656, 52, 128, 17920, 32000, "bf16"),
}


@dataclass(frozen=True)
class Workload:
    name: str
    model: str
    prefix_len: int
    n_nodes: int
    max_levels: int
    branching: str  # "binary" | "uniform4" | "geometric4" | "chain" | "star"


WORKLOADS: Dict[str, Workload] = {
    "C1": Workload("C1", "tiny", 32, 15, 4, "binary"),
    "C2": Workload("C2", "7b", 512, 32, 8, "uniform4"),
    "C3": Workload("C3", "13b", 1024, 64, 10, "geometric4"),
    "C5": Workload("C5", "30b", 2048, 128, 12, "uniform4"),
}


def shrink(cfg: ModelConfig, n_layers: int) -> ModelConfig:
    """Same widths, fewer layers (parity cases the oracle finishes quickly)."""
    return replace(cfg, n_layers=n_layers, name=f"{cfg.name}-L{n_layers}")


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([MASTER_SEED, *key])))


def _to_dtype(a: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(a)
    return t if dtype == "f32" else t.to(torch.bfloat16)


def tensor_shape(cfg: ModelConfig, name: str):
    d, f, v = cfg.d_model, cfg.d_ffn, cfg.vocab
    return {
        "tok_embed": (v, d), "lm_head": (v, d), "final_norm": (d,),
        "attn_norm": (d,), "ffn_norm": (d,),
        "wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d),
        "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f),
    }[name]


_GEN_BLOCK_ROWS = 1024      # rows per independent random stream of a weight matrix
_gen_pool = None


def _gen_block(shape, key, r0, r1, out):
    g = _rng(*key, r0 // _GEN_BLOCK_ROWS)
    a = g.standard_normal((r1 - r0, *shape[1:]), dtype=np.float32)
    a *= np.float32(0.02)
    out[r0:r1] = a


def gen_tensor(cfg: ModelConfig, name: str, layer: int = -1, seed: int = 0) -> torch.Tensor:
    """One weight tensor, row-major [out][in], in the config's storage dtype (CPU). A matrix is drawn
    in blocks of 1024 rows, each from its own stream keyed by (seed, layer, tensor, block), so that
    the blocks of a large matrix can be drawn on all host cores at once."""
    global _gen_pool
    shape = tensor_shape(cfg, name)
    if name.endswith("norm"):
        return _to_dtype(np.ones(shape, dtype=np.float32), cfg.dtype)
    key = (seed, layer + 1, _TID[name])
    out = np.empty(shape, dtype=np.float32)
    blocks = [(r0, min(shape[0], r0 + _GEN_BLOCK_ROWS)) for r0 in range(0, shape[0], _GEN_BLOCK_ROWS)]
    if len(blocks) == 1:
        _gen_block(shape, key, 0, shape[0], out)
    else:
        if _gen_pool is None:
            import os
            from concurrent.futures import ThreadPoolExecutor
            _gen_pool = ThreadPoolExecutor(len(os.sched_getaffinity(0)))
        list(_gen_pool.map(lambda b: _gen_block(shape, key, b[0], b[1], out), blocks))
    return _to_dtype(out, cfg.dtype)


def gen_layer(cfg: ModelConfig, layer: int, seed: int = 0) -> Dict[str, torch.Tensor]:
    return {n: gen_tensor(cfg, n, layer, seed) for n in LAYER_TENSORS}


def gen_globals(cfg: ModelConfig, seed: int = 0) -> Dict[str, torch.Tensor]:
    return {n: gen_tensor(cfg, n, -1, seed) for n in ("tok_embed", "final_norm", "lm_head")}


def gen_tensor_device(cfg: ModelConfig, name: str, layer: int, device, seed: int = 0) -> torch.Tensor:
    """Same recipe drawn by the device's own generator (bench only: filling 13-65 GB
    from host cores would dominate the run). Values differ from gen_tensor's."""
    shape = tensor_shape(cfg, name)
    if name.endswith("norm"):
        return torch.ones(shape, dtype=cfg.torch_dtype, device=device)
    g = torch.Generator(device=device)
    g.manual_seed((MASTER_SEED * 1000003 + seed * 10007 + (layer + 1) * 101 + _TID[name]) & 0x7FFFFFFF)
    out = torch.empty(shape, dtype=cfg.torch_dtype, device=device)
    # draw in row chunks so the fp32 staging buffer stays small
    rows = shape[0]
    step = max(1, (64 << 20) // max(1, int(np.prod(shape[1:]))))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        out[r0:r1] = (torch.randn((r1 - r0, *shape[1:]), generator=g, device=device, dtype=torch.float32) * 0.02).to(cfg.torch_dtype)
    return out


def gen_prefix_kv(cfg: ModelConfig, layer: int, prefix_len: int, seed: int = 0):
    """Synthetic prefix cache rows of one layer: K, V of shape [H][P][hd] ~ N(0,1)."""
    out = []
    for name in ("prefix_k", "prefix_v"):
        g = _rng(seed, layer + 1, _TID[name])
        a = g.standard_normal((cfg.n_heads, prefix_len, cfg.head_dim), dtype=np.float32)
        out.append(_to_dtype(a, cfg.dtype))
    return out[0], out[1]


def gen_prefix_tokens(cfg: ModelConfig, prefix_len: int, seed: int = 0) -> np.ndarray:
    return _rng(seed, 0, 40).integers(0, cfg.vocab, size=prefix_len, dtype=np.int32)


def gen_tokens(cfg: ModelConfig, n: int, seed: int = 0) -> np.ndarray:
    return _rng(seed, 0, 41).integers(0, cfg.vocab, size=n, dtype=np.int32)


# --------------------------------------------------------------------------- trees

def tree_binary(levels: int) -> np.ndarray:
    n = (1 << levels) - 1
    p = np.empty(n, dtype=np.int32)
    p[0] = -1
    for i in range(1, n):
        p[i] = (i - 1) // 2
    return p


def tree_chain(n: int) -> np.ndarray:
    return np.arange(-1, n - 1, dtype=np.int32)


def tree_star(n: int) -> np.ndarray:
    p = np.zeros(n, dtype=np.int32)
    p[0] = -1
    return p


def tree_random(n: int, max_levels: int, branching: str, seed: int = 0) -> np.ndarray:
    """Grow a tree from a frontier: pick a frontier node uniformly, draw its number of
    children b, attach min(b, remaining) children when the node's level allows,
    otherwise drop it. Nodes are numbered in creation order so parent_idx[i] < i."""
    g = _rng(seed, 0, 50)
    parent = [-1]
    level = [1]
    frontier = [0]
    while len(parent) < n:
        if not frontier:
            # every frontier node sat on the last level: restart from the shallowest leaf-capable nodes
            frontier = [i for i in range(len(parent)) if level[i] < max_levels]
            if not frontier:
                raise ValueError("tree cannot reach n nodes within max_levels")
        k = int(g.integers(0, len(frontier)))
        node = frontier.pop(k)
        if level[node] >= max_levels:
            continue
        if branching == "uniform4":
            b = int(g.integers(1, 5))
        elif branching == "geometric4":
            b = min(4, int(g.geometric(0.5)))
        else:
            raise ValueError(branching)
        b = min(b, n - len(parent))
        for _ in range(b):
            parent.append(node)
            level.append(level[node] + 1)
            frontier.append(len(parent) - 1)
    return np.asarray(parent, dtype=np.int32)


def gen_tree(w: Workload, seed: int = 0) -> np.ndarray:
    if w.branching == "binary":
        return tree_binary(w.max_levels)
    if w.branching == "chain":
        return tree_chain(w.n_nodes)
    if w.branching == "star":
        return tree_star(w.n_nodes)
    return tree_random(w.n_nodes, w.max_levels, w.branching, seed)


def plant_tokens(parent_idx: np.ndarray, tokens: np.ndarray, argmax: np.ndarray, seed: int = 0,
                 prob: float = 0.7) -> np.ndarray:
    """"Planted" variant: with probability `prob` per node that has children, overwrite
    one child's token with the supplied argmax of its parent, so that acceptance and
    compaction have something to accept. `argmax` is data handed in by the caller."""
    g = _rng(seed, 0, 60)
    n = len(parent_idx)
    out = tokens.copy()
    children: List[List[int]] = [[] for _ in range(n)]
    for i in range(1, n):
        children[int(parent_idx[i])].append(i)
    for i in range(n):
        if children[i] and g.random() < prob:
            c = children[i][int(g.integers(0, len(children[i])))]
            out[c] = argmax[i]
    return out


def relabel_tree(parent_idx: np.ndarray, seed: int = 0):
    """A different topological numbering of the same tree. Returns (new_parent, perm)
    with perm[new] = old."""
    g = _rng(seed, 0, 70)
    n = len(parent_idx)
    children: List[List[int]] = [[] for _ in range(n)]
    for i in range(1, n):
        children[int(parent_idx[i])].append(i)
    order: List[int] = []
    ready = [0]
    while ready:
        k = int(g.integers(0, len(ready)))
        node = ready.pop(k)
        order.append(node)
        ready.extend(children[node])
    new_of_old = {o: i for i, o in enumerate(order)}
    newp = np.asarray([-1 if parent_idx[o] < 0 else new_of_old[int(parent_idx[o])] for o in order], dtype=np.int32)
    return newp, np.asarray(order, dtype=np.int32)


def gen_attention_inputs(n_heads: int, head_dim: int, prefix_len: int, n_nodes: int, seed: int = 0,
                         dtype: str = "bf16"):
    """Attention-only case: q [N][H][hd]; K, V [H][P+N][hd], all ~ N(0,1)."""
    g = _rng(seed, prefix_len, n_nodes, _TID["q"])
    q = g.standard_normal((n_nodes, n_heads, head_dim), dtype=np.float32)
    k = g.standard_normal((n_heads, prefix_len + n_nodes, head_dim), dtype=np.float32)
    v = g.standard_normal((n_heads, prefix_len + n_nodes, head_dim), dtype=np.float32)
    return _to_dtype(q, dtype), _to_dtype(k, dtype), _to_dtype(v, dtype)
