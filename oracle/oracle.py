"""ctypes front end of the CPU oracle (oracle.c, sequential.c).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
cpu_baseline / reference leg may import this. It holds argument marshalling and
the layer-streaming loop; the arithmetic is in the two C files.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Callable, Dict, Iterable, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liboracle.so")
_SRCS = [os.path.join(_HERE, "oracle.c"), os.path.join(_HERE, "sequential.c")]
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over output rows)."""
    newest = max(os.path.getmtime(s) for s in _SRCS)
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < newest:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, *_SRCS, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


class _Cfg(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("d_model", C.c_int), ("n_heads", C.c_int), ("head_dim", C.c_int),
                ("d_ffn", C.c_int), ("vocab", C.c_int), ("rms_eps", C.c_double), ("rope_base", C.c_double)]


class _SeqLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops use: the cores this process may run on."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def _cfg(cfg) -> _Cfg:
    return _Cfg(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.d_ffn, cfg.vocab,
                float(cfg.rms_eps), float(cfg.rope_base))


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _f32(t) -> np.ndarray:
    """Weights as contiguous fp32 (bf16 widens exactly)."""
    if hasattr(t, "detach"):
        t = t.detach().float().cpu().numpy()
    return np.ascontiguousarray(t, dtype=np.float32)


def _f64(t) -> np.ndarray:
    if hasattr(t, "detach"):
        t = t.detach().double().cpu().numpy()
    return np.ascontiguousarray(t, dtype=np.float64)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


# ------------------------------------------------------------------ single steps

def tree_prep(parent_idx, prefix_len: int):
    p = _i32(parent_idx)
    n = len(p)
    depth = np.zeros(n, np.int32)
    pos = np.zeros(n, np.int32)
    anc = np.zeros((n, n), np.uint8)
    st = lib().orc_tree_prep(_p(p), n, int(prefix_len), _p(depth), _p(pos), _p(anc))
    return st, depth, pos, anc


def rmsnorm(x, g, eps: float):
    x = _f64(x); g = _f32(g)
    out = np.empty_like(x)
    lib().orc_rmsnorm(_p(x), _p(g), x.shape[0], x.shape[1], C.c_double(eps), _p(out))
    return out


def linear(W, x):
    W = _f32(W); x = _f64(x)
    y = np.empty((x.shape[0], W.shape[0]), np.float64)
    lib().orc_linear(_p(W), W.shape[0], W.shape[1], _p(x), x.shape[0], _p(y))
    return y


def rope(v, pos, n_heads: int, hd: int, base: float):
    v = _f64(v).copy(); pos = _i32(pos)
    lib().orc_rope(_p(v), _p(pos), v.shape[0], n_heads, hd, C.c_double(base))
    return v


def tree_attention(q, prefix_k, prefix_v, tree_k, tree_v, anc, n_heads: int, hd: int):
    """q, tree_k, tree_v [n][H*hd]; prefix_k, prefix_v [H][P][hd]; anc [n][n] -> o [n][H*hd]."""
    q = _f64(q); pk = _f64(prefix_k); pv = _f64(prefix_v); tk = _f64(tree_k); tv = _f64(tree_v)
    anc = np.ascontiguousarray(anc, dtype=np.uint8)
    n = q.shape[0]
    P = pk.shape[1]
    o = np.empty_like(q)
    lib().orc_tree_attention(_p(q), _p(pk), _p(pv), P, _p(tk), _p(tv), _p(anc), n, n_heads, hd, _p(o))
    return o


def argmax(logits):
    lg = _f64(logits)
    out = np.zeros(lg.shape[0], np.int32)
    lib().orc_argmax(_p(lg), lg.shape[0], lg.shape[1], _p(out))
    return out


@dataclass
class Acceptance:
    path: np.ndarray
    accepted_len: int
    next_token: int
    n_correct: int
    n_all: int
    rectified: int


def accept(parent_idx, tokens, argmax_) -> Acceptance:
    p = _i32(parent_idx); t = _i32(tokens); a = _i32(argmax_)
    n = len(p)
    path = np.zeros(n, np.int32)
    res = np.zeros(6, np.int32)
    lib().orc_accept(_p(p), _p(t), _p(a), n, _p(path), _p(res))
    return Acceptance(path[: res[0]].copy(), int(res[0]), int(res[1]), int(res[2]), int(res[3]), int(res[4]))


def compact(prefix, tree, path, n_heads: int, hd: int):
    """prefix [H][P][hd], tree [n][H*hd] -> [H][P+len][hd]"""
    prefix = _f64(prefix); tree = _f64(tree); path = _i32(path)
    P = prefix.shape[1]
    out = np.empty((n_heads, P + len(path), hd), np.float64)
    lib().orc_compact(_p(prefix), _p(tree), P, n_heads, hd, _p(path), len(path), _p(out))
    return out


# ------------------------------------------------------------------ whole pass

@dataclass
class PassResult:
    status: int
    depth: np.ndarray
    pos: np.ndarray
    anc: np.ndarray
    logits: Optional[np.ndarray] = None      # [n][V] fp64
    argmax: Optional[np.ndarray] = None
    acceptance: Optional[Acceptance] = None
    tree_k: Optional[list] = None            # per layer [n][d] fp64 (post-rotation)
    tree_v: Optional[list] = None
    new_prefix_len: int = 0


def verify_tree(cfg, globals_: Dict, layer_fn: Callable[[int], Dict], prefix_fn: Callable[[int], Tuple],
                prefix_len: int, tokens, parent_idx, keep_kv: bool = True,
                layer_times: Optional[list] = None) -> PassResult:
    """One verification pass, layer-streamed: `layer_fn(l)` returns layer l's weight
    dict and `prefix_fn(l)` its prefix (K, V) as [H][P][hd]; each is dropped after
    use so that no more than one layer is resident."""
    import time
    c = _cfg(cfg)
    tokens = _i32(tokens); parent_idx = _i32(parent_idx)
    n = len(tokens)
    st, depth, pos, anc = tree_prep(parent_idx, prefix_len)
    res = PassResult(st, depth, pos, anc, new_prefix_len=prefix_len)
    if st:
        return res
    x = np.zeros((n, cfg.d_model), np.float64)
    E = _f32(globals_["tok_embed"])
    st = lib().orc_embed(C.byref(c), _p(E), _p(tokens), n, _p(x))
    if st:
        res.status = st
        return res
    tks, tvs = [], []
    for l in range(cfg.n_layers):
        w = {k: _f32(v) for k, v in layer_fn(l).items()}
        pk, pv = prefix_fn(l)
        pk = _f64(pk).reshape(cfg.n_heads, prefix_len, cfg.head_dim)
        pv = _f64(pv).reshape(cfg.n_heads, prefix_len, cfg.head_dim)
        tk = np.empty((n, cfg.d_model), np.float64)
        tv = np.empty((n, cfg.d_model), np.float64)
        t0 = time.perf_counter()
        lib().orc_layer(C.byref(c), _p(w["attn_norm"]), _p(w["wq"]), _p(w["wk"]), _p(w["wv"]), _p(w["wo"]),
                        _p(w["ffn_norm"]), _p(w["w_gate"]), _p(w["w_up"]), _p(w["w_down"]),
                        _p(pk), _p(pv), int(prefix_len), _p(pos), _p(anc), n, _p(x), _p(tk), _p(tv))
        if layer_times is not None:
            layer_times.append(time.perf_counter() - t0)
        if keep_kv:
            tks.append(tk); tvs.append(tv)
        del w, pk, pv
    logits = np.empty((n, cfg.vocab), np.float64)
    fn = _f32(globals_["final_norm"]); lm = _f32(globals_["lm_head"])
    t0 = time.perf_counter()
    lib().orc_head(C.byref(c), _p(fn), _p(lm), _p(x), n, _p(logits))
    if layer_times is not None:
        layer_times.append(time.perf_counter() - t0)
    res.logits = logits
    res.argmax = argmax(logits)
    res.acceptance = accept(parent_idx, tokens, res.argmax)
    res.tree_k, res.tree_v = tks, tvs
    res.new_prefix_len = prefix_len + res.acceptance.accepted_len
    return res


# ------------------------------------------------------------------ sequential decoder

class SequentialDecoder:
    """Ordinary one-token-at-a-time decoding with a causal KV cache (sequential.c)."""

    def __init__(self, cfg, globals_: Dict, layers: Iterable[Dict], max_seq: int):
        self.cfg = cfg
        self.c = _cfg(cfg)
        self.max_seq = max_seq
        self.E = _f32(globals_["tok_embed"]); self.fn = _f32(globals_["final_norm"]); self.lm = _f32(globals_["lm_head"])
        self._keep = []
        arr = (_SeqLayer * cfg.n_layers)()
        for l, w in enumerate(layers):
            w32 = {k: _f32(v) for k, v in w.items()}
            self._keep.append(w32)
            for k, v in w32.items():
                setattr(arr[l], k, v.ctypes.data)
        self.layers = arr
        self.kc = np.zeros((cfg.n_layers, max_seq, cfg.d_model), np.float64)
        self.vc = np.zeros((cfg.n_layers, max_seq, cfg.d_model), np.float64)
        self.t = 0

    def step(self, token: int) -> np.ndarray:
        logits = np.empty(self.cfg.vocab, np.float64)
        st = lib().seq_decode_step(C.byref(self.c), _p(self.E), self.layers, _p(self.fn), _p(self.lm),
                                   _p(self.kc), _p(self.vc), self.max_seq, self.t, int(token), _p(logits))
        if st:
            raise ValueError("seq_decode_step: bad token or position")
        self.t += 1
        return logits

    def truncate(self, t: int):
        self.t = t

    def cache_heads(self, layer: int, upto: int):
        """Rows 0..upto-1 of one layer's cache as ([H][upto][hd], same for V)."""
        H, hd = self.cfg.n_heads, self.cfg.head_dim
        k = self.kc[layer, :upto].reshape(upto, H, hd).transpose(1, 0, 2)
        v = self.vc[layer, :upto].reshape(upto, H, hd).transpose(1, 0, 2)
        return np.ascontiguousarray(k), np.ascontiguousarray(v)


def tree_confidence(branch_conf) -> float:
    """Sec. 3.3: T_c = max over branches of the cumulative confidence."""
    c = np.ascontiguousarray(branch_conf, dtype=np.float64)
    f = lib().orc_tree_confidence
    f.restype = C.c_double
    return float(f(_p(c), C.c_int(len(c))))


def alpha_update(alpha: float, n_correct: int, n_all: int, t_c: float) -> float:
    """Eq. 3: the self-adaptive fallback threshold after one verification."""
    f = lib().orc_alpha_update
    f.restype = C.c_double
    f.argtypes = [C.c_double, C.c_int, C.c_int, C.c_double]
    return float(f(alpha, n_correct, n_all, t_c))


def topk_softmax(logits: np.ndarray, k: int):
    """Softmax of every row and its k largest entries (descending, ties to the lower id): (ids, probs)."""
    lg = np.ascontiguousarray(logits, dtype=np.float64)
    n, vocab = lg.shape
    ids = np.zeros((n, k), np.int32)
    probs = np.zeros((n, k), np.float64)
    lib().orc_topk_softmax(_p(lg), C.c_int(n), C.c_int(vocab), C.c_int(k), _p(ids), _p(probs))
    return ids, probs


def tree_branches(parent, node_conf):
    """Sec. 3.2: the root-to-leaf branches of a tree: (leaf ids, cumulative confidences, draft tokens per branch)."""
    par = np.ascontiguousarray(parent, dtype=np.int32)
    conf = np.ascontiguousarray(node_conf, dtype=np.float64)
    n = len(par)
    leaf = np.zeros(n, np.int32)
    cum = np.zeros(n, np.float64)
    length = np.zeros(n, np.int32)
    f = lib().orc_tree_branches
    f.restype = C.c_int
    nb = int(f(_p(par), _p(conf), C.c_int(n), _p(leaf), _p(cum), _p(length)))
    return leaf[:nb].copy(), cum[:nb].copy(), length[:nb].copy()


def branch_pacer(cum_conf, branch_len, m_tokens: float):
    """Eq. 1-2: (f(x) for every branch, the branch that gets the next token)."""
    c = np.ascontiguousarray(cum_conf, dtype=np.float64)
    t = np.ascontiguousarray(branch_len, dtype=np.int32)
    out = np.zeros(len(c), np.float64)
    f = lib().orc_branch_pacer
    f.restype = C.c_int
    nxt = int(f(_p(c), _p(t), C.c_int(len(c)), C.c_double(float(m_tokens)), _p(out)))
    return out, nxt


INT4_GROUP = 64


def quantize_int4(w, group: int = INT4_GROUP):
    """Sec. 4.1 (INT4 weights): symmetric group quantisation with power-of-two scales.
    w [rows][cols] -> (q int8 [rows][cols] in [-8, 7], e int8 [rows][cols / group])."""
    w = _f32(w)
    rows, cols = w.shape
    assert cols % group == 0
    q = np.zeros((rows, cols), np.int8)
    e = np.zeros((rows, cols // group), np.int8)
    lib().orc_quantize_int4(_p(w), C.c_int(rows), C.c_int(cols), C.c_int(group), _p(q), _p(e))
    return q, e


def dequantize_int4(q, e, group: int = INT4_GROUP) -> np.ndarray:
    """q * 2^e as fp32 (every value is exactly representable in bf16)."""
    q = np.ascontiguousarray(q, dtype=np.int8)
    e = np.ascontiguousarray(e, dtype=np.int8)
    rows, cols = q.shape
    w = np.zeros((rows, cols), np.float32)
    lib().orc_dequantize_int4(_p(q), _p(e), C.c_int(rows), C.c_int(cols), C.c_int(group), _p(w))
    return w


def int4_weights(layer: Dict, group: int = INT4_GROUP) -> Dict:
    """The layer a quantised model computes with: every matrix replaced by its dequantised INT4 form
    (norm gains stay as they are)."""
    out = {}
    for k, v in layer.items():
        if k.endswith("norm"):
            out[k] = v
        else:
            out[k] = dequantize_int4(*quantize_int4(v, group), group)
    return out
