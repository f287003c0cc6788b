"""Thin ctypes binding of libllmcad.so: argument marshalling only.

Every step of the verification pass runs in the library's CUDA kernels; torch is
used here for device memory and streams. There is no fallback: importing works
anywhere, but any call needs the built library and a CUDA device and fails
loudly otherwise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# LLMCAD_LIB selects another build of the same library (the debug build with device-side checks)
LIB_PATH = os.environ.get("LLMCAD_LIB") or os.path.join(_HERE, "libllmcad.so")
MAX_TREE = 128

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CAPACITY, ERR_CUDA = 0, -1, -2, -3, -4
ERR_BAD_TREE, ERR_BAD_TOKEN, ERR_TIMEOUT, ERR_NAN, ERR_CHECK = 1, 2, 3, 4, 5
F32, BF16 = 0, 1
FLAG_SIMT_GEMM, FLAG_SIMT_ATTN, FLAG_T5_ATTN, FLAG_MMA_ATTN, FLAG_INT4_WEIGHTS = 1, 2, 4, 8, 16
S_ACCEPTED_LEN, S_NEXT_TOKEN, S_NEW_PREFIX_LEN, S_N_CORRECT, S_N_ALL, S_RECTIFIED, S_STATUS = range(7)

EXPORTS = [
    "llmcad_version", "llmcad_strerror", "llmcad_last_cuda_error", "llmcad_create", "llmcad_destroy",
    "llmcad_kv_cache_bytes", "llmcad_packed_weight_bytes", "llmcad_pack_layer", "llmcad_pack_globals",
    "llmcad_verify_tree", "llmcad_verify_tree_host", "llmcad_prefill", "llmcad_tree_prep",
    "llmcad_accept_compact", "llmcad_tree_attention", "llmcad_skinny_gemm", "llmcad_launch_count",
    "llmcad_last_status", "llmcad_set_kernel_timing", "llmcad_get_kernel_timing", "llmcad_set_gemm_trace", "llmcad_tiled_weight_bytes", "llmcad_tile_weight", "llmcad_skinny_gemm_tiled", "llmcad_tree_attention_noalloc", "llmcad_noalloc_last_error",
    "llmcad_tree_confidence", "llmcad_update_threshold", "llmcad_extend_tree", "llmcad_tree_branches", "llmcad_branch_pacer",
    "llmcad_set_wait_limit_ns", "llmcad_selftest_wait_timeout",
    "llmcad_quantize_int4", "llmcad_tiled_weight_int4_bytes", "llmcad_tile_weight_int4", "llmcad_skinny_gemm_tiled_int4",
    "llmcad_probe_bulk_copy", "llmcad_probe_mma_sync",
]


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("d_ffn", C.c_int32), ("vocab", C.c_int32), ("max_seq", C.c_int32), ("max_tree", C.c_int32),
                ("rms_eps", C.c_float), ("rope_base", C.c_float), ("dtype", C.c_int32), ("flags", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class GlobalWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tok_embed", "final_norm", "lm_head")]


class Result(C.Structure):
    _fields_ = [("logits", C.c_void_p), ("argmax", C.c_void_p), ("accepted_path", C.c_void_p), ("scalars", C.c_void_p)]


class LlmcadError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().llmcad_strerror(code).decode()
        if code == ERR_CUDA:
            msg += " (" + lib().llmcad_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {msg} [{code}]")


_lib = None


def lib():
    """The loaded C-ABI library. Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2309_04255_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        L.llmcad_version.restype = C.c_int
        L.llmcad_strerror.restype = C.c_char_p
        L.llmcad_strerror.argtypes = [C.c_int]
        L.llmcad_last_cuda_error.restype = C.c_char_p
        L.llmcad_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
        L.llmcad_destroy.argtypes = [vp]
        L.llmcad_destroy.restype = None
        L.llmcad_kv_cache_bytes.argtypes = [C.POINTER(Config)]
        L.llmcad_kv_cache_bytes.restype = sz
        L.llmcad_packed_weight_bytes.argtypes = [C.POINTER(Config)]
        L.llmcad_packed_weight_bytes.restype = sz
        L.llmcad_pack_layer.argtypes = [vp, i32, C.POINTER(LayerWeights), vp, vp]
        L.llmcad_pack_globals.argtypes = [vp, C.POINTER(GlobalWeights), vp, vp]
        L.llmcad_verify_tree.argtypes = [vp, vp, vp, i32, vp, vp, i32, C.POINTER(Result), vp]
        L.llmcad_verify_tree_host.argtypes = [vp, vp, vp, i32, vp, vp, i32, C.POINTER(Result), vp]
        L.llmcad_prefill.argtypes = [vp, vp, vp, i32, vp, i32, vp, vp]
        L.llmcad_tree_prep.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
        L.llmcad_accept_compact.argtypes = [vp, vp, i32, vp, vp, vp, i32, vp, vp, vp]
        L.llmcad_tree_attention.argtypes = [vp, vp, vp, vp, i32, i32, vp, i32, vp, vp]
        L.llmcad_skinny_gemm.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
        L.llmcad_launch_count.argtypes = [vp]
        L.llmcad_launch_count.restype = C.c_int64
        L.llmcad_last_status.argtypes = [vp, vp]
        L.llmcad_set_gemm_trace.argtypes = [vp, vp, i32]
        L.llmcad_tiled_weight_bytes.argtypes = [i32, i32]
        L.llmcad_tiled_weight_bytes.restype = sz
        L.llmcad_tile_weight.argtypes = [vp, i32, i32, vp, vp]
        L.llmcad_skinny_gemm_tiled.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
        L.llmcad_tree_attention_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, vp, i32, vp, vp, vp]
        L.llmcad_noalloc_last_error.restype = C.c_char_p
        L.llmcad_extend_tree.argtypes = [vp, vp, vp, i32, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp]
        L.llmcad_set_kernel_timing.argtypes = [vp, i32]
        L.llmcad_get_kernel_timing.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.llmcad_quantize_int4.argtypes = [vp, i32, i32, vp, vp, vp]
        L.llmcad_tiled_weight_int4_bytes.argtypes = [i32, i32]
        L.llmcad_tiled_weight_int4_bytes.restype = sz
        L.llmcad_tile_weight_int4.argtypes = [vp, i32, i32, vp, vp]
        L.llmcad_skinny_gemm_tiled_int4.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
        L.llmcad_set_wait_limit_ns.argtypes = [vp, C.c_uint64]
        L.llmcad_selftest_wait_timeout.argtypes = [vp, vp]
        L.llmcad_probe_bulk_copy.argtypes = [vp, sz, i32, i32, vp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.llmcad_probe_mma_sync.argtypes = [i32, i32, vp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != OK:
        raise LlmcadError(code, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


def make_config(cfg, max_seq: int, max_tree: int = MAX_TREE, flags: int = 0) -> Config:
    return Config(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.d_ffn, cfg.vocab, max_seq, max_tree,
                  cfg.rms_eps, cfg.rope_base, F32 if cfg.dtype == "f32" else BF16, flags)


class Verifier:
    """One context + its packed weights and KV cache (device memory held as torch tensors)."""

    def __init__(self, cfg, max_seq: int, max_tree: int = MAX_TREE, flags: int = 0, device="cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("llmcad needs a CUDA device; there is no CPU path")
        self.cfg = cfg
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.c = make_config(cfg, max_seq, max_tree, flags)
        self.max_seq, self.max_tree = max_seq, max_tree
        h = C.c_void_p()
        _check(lib().llmcad_create(C.byref(self.c), C.byref(h)), "llmcad_create")
        self.ctx = h
        self.packed = torch.empty(lib().llmcad_packed_weight_bytes(C.byref(self.c)), dtype=torch.uint8, device=self.device)
        self.kv = torch.zeros(lib().llmcad_kv_cache_bytes(C.byref(self.c)), dtype=torch.uint8, device=self.device)
        self.tdtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16

    def close(self):
        if getattr(self, "ctx", None):
            torch.cuda.synchronize()
            lib().llmcad_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- weights
    def pack_layer(self, layer: int, w: Dict[str, torch.Tensor]):
        dev = {k: v.to(self.device, self.tdtype).contiguous() for k, v in w.items()}
        lw = LayerWeights(**{k: dev[k].data_ptr() for k in dev})
        _check(lib().llmcad_pack_layer(self.ctx, layer, C.byref(lw), self.packed.data_ptr(), _stream()), "llmcad_pack_layer")
        torch.cuda.current_stream().synchronize()  # sources go out of scope here

    def pack_globals(self, w: Dict[str, torch.Tensor]):
        dev = {k: v.to(self.device, self.tdtype).contiguous() for k, v in w.items()}
        gw = GlobalWeights(**{k: dev[k].data_ptr() for k in dev})
        _check(lib().llmcad_pack_globals(self.ctx, C.byref(gw), self.packed.data_ptr(), _stream()), "llmcad_pack_globals")
        torch.cuda.current_stream().synchronize()

    # ---- cache views
    def kv_view(self) -> torch.Tensor:
        """[L][2][H][max_seq][hd] view of the cache in the model dtype."""
        c = self.cfg
        return self.kv.view(self.tdtype).view(c.n_layers, 2, c.n_heads, self.max_seq, c.head_dim)

    # ---- the pass
    def new_outputs(self, n: int, want_logits: bool = True):
        dev = self.device
        return {
            "logits": torch.empty((n, self.cfg.vocab), dtype=torch.float32, device=dev) if want_logits else None,
            "argmax": torch.empty(n, dtype=torch.int32, device=dev),
            "accepted_path": torch.full((self.max_tree,), -1, dtype=torch.int32, device=dev),
            "scalars": torch.zeros(8, dtype=torch.int32, device=dev),
        }

    def verify_tree(self, prefix_len: int, tokens: torch.Tensor, parent: torch.Tensor, out=None, want_logits=True):
        n = tokens.numel()
        out = out or self.new_outputs(n, want_logits)
        r = Result(_ptr(out["logits"]), _ptr(out["argmax"]), _ptr(out["accepted_path"]), _ptr(out["scalars"]))
        _check(lib().llmcad_verify_tree(self.ctx, self.packed.data_ptr(), self.kv.data_ptr(), prefix_len, _ptr(tokens),
                                        _ptr(parent), n, C.byref(r), _stream()), "llmcad_verify_tree")
        return out

    def extend_tree(self, prefix_len: int, tokens: torch.Tensor, parent: torch.Tensor, n_old: int, top_k: int = 4,
                    want_logits: bool = True):
        """Decoder forward of the tree nodes n_old.. (the K/V of the first n_old nodes are in the cache):
        returns logits [n_new][vocab] (or None), top-k ids and probabilities [n_new][top_k], status."""
        n_tree = tokens.numel()
        n_new = n_tree - n_old
        dev = self.device
        out = {
            "logits": torch.empty((n_new, self.cfg.vocab), dtype=torch.float32, device=dev) if want_logits else None,
            "topk_ids": torch.empty((n_new, max(top_k, 1)), dtype=torch.int32, device=dev),
            "topk_probs": torch.empty((n_new, max(top_k, 1)), dtype=torch.float32, device=dev),
            "status": torch.zeros(1, dtype=torch.int32, device=dev),
        }
        _check(lib().llmcad_extend_tree(self.ctx, _ptr(self.packed), _ptr(self.kv), prefix_len, _ptr(tokens), _ptr(parent),
                                        n_old, n_tree, top_k, _ptr(out["logits"]), _ptr(out["topk_ids"]),
                                        _ptr(out["topk_probs"]), _ptr(out["status"]), _stream()), "llmcad_extend_tree")
        return out

    def verify_tree_host(self, prefix_len: int, tokens: torch.Tensor, parent: torch.Tensor, out):
        """tokens/parent and the tensors of `out` live in (pinned) host memory."""
        n = tokens.numel()
        lg = out.get("logits")
        r = Result(lg.data_ptr() if lg is not None else None, out["argmax"].data_ptr(),
                   out["accepted_path"].data_ptr(), out["scalars"].data_ptr())
        _check(lib().llmcad_verify_tree_host(self.ctx, self.packed.data_ptr(), self.kv.data_ptr(), prefix_len,
                                             tokens.data_ptr(), parent.data_ptr(), n, C.byref(r), _stream()),
               "llmcad_verify_tree_host")
        return out

    def prefill(self, prefix_len: int, tokens: torch.Tensor, want_logits: bool = False):
        lg = torch.empty(self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        _check(lib().llmcad_prefill(self.ctx, self.packed.data_ptr(), self.kv.data_ptr(), prefix_len, _ptr(tokens),
                                    tokens.numel(), _ptr(lg), _stream()), "llmcad_prefill")
        return lg

    # ---- single steps
    def accept_compact(self, prefix_len: int, tokens, parent, argmax, compact: bool = True):
        n = tokens.numel()
        path = torch.full((self.max_tree,), -1, dtype=torch.int32, device=self.device)
        scalars = torch.zeros(8, dtype=torch.int32, device=self.device)
        _check(lib().llmcad_accept_compact(self.ctx, self.kv.data_ptr() if compact else None, prefix_len, _ptr(tokens),
                                           _ptr(parent), _ptr(argmax), n, _ptr(path), _ptr(scalars), _stream()),
               "llmcad_accept_compact")
        return path, scalars

    def tree_attention(self, q, k, v, prefix_len: int, parent, o=None):
        """q [n][H][hd]; k, v [H][kv_stride][hd]; o (optional) receives the result."""
        n = q.shape[0]
        o = torch.empty_like(q) if o is None else o
        _check(lib().llmcad_tree_attention(self.ctx, _ptr(q), _ptr(k), _ptr(v), k.shape[1], prefix_len, _ptr(parent), n,
                                           _ptr(o), _stream()), "llmcad_tree_attention")
        return o

    def skinny_gemm(self, w, x):
        n, n_in = x.shape
        n_out = w.shape[0]
        y = torch.empty((n, n_out), dtype=torch.float32, device=self.device)
        _check(lib().llmcad_skinny_gemm(self.ctx, _ptr(w), _ptr(x), _ptr(y), n_out, n_in, n, _stream()), "llmcad_skinny_gemm")
        return y

    def tile_weight(self, w):
        """Row-major bf16 [n_out][n_in] -> the tiled layout the tensor-core GEMM streams."""
        n_out, n_in = w.shape
        t = torch.empty(lib().llmcad_tiled_weight_bytes(n_out, n_in), dtype=torch.uint8, device=self.device)
        _check(lib().llmcad_tile_weight(_ptr(w), n_out, n_in, _ptr(t), _stream()), "llmcad_tile_weight")
        return t

    def skinny_gemm_tiled(self, w_tiled, n_out, x):
        n, n_in = x.shape
        y = torch.empty((n, n_out), dtype=torch.float32, device=self.device)
        _check(lib().llmcad_skinny_gemm_tiled(self.ctx, _ptr(w_tiled), _ptr(x), _ptr(y), n_out, n_in, n, _stream()),
               "llmcad_skinny_gemm_tiled")
        return y

    def tile_weight_int4(self, w):
        """Row-major bf16 [n_out][n_in] -> INT4 codes and group exponents in the layout the GEMM streams."""
        n_out, n_in = w.shape
        t = torch.empty(lib().llmcad_tiled_weight_int4_bytes(n_out, n_in), dtype=torch.uint8, device=self.device)
        _check(lib().llmcad_tile_weight_int4(_ptr(w), n_out, n_in, _ptr(t), _stream()), "llmcad_tile_weight_int4")
        return t

    def skinny_gemm_tiled_int4(self, w_tiled, n_out, x):
        n, n_in = x.shape
        y = torch.empty((n, n_out), dtype=torch.float32, device=self.device)
        _check(lib().llmcad_skinny_gemm_tiled_int4(self.ctx, _ptr(w_tiled), _ptr(x), _ptr(y), n_out, n_in, n, _stream()),
               "llmcad_skinny_gemm_tiled_int4")
        return y

    def last_status(self) -> int:
        return lib().llmcad_last_status(self.ctx, _stream())

    def set_gemm_trace(self, buf: Optional[torch.Tensor]):
        """buf: int64 cuda tensor [capacity][256][16] or None."""
        _check(lib().llmcad_set_gemm_trace(self.ctx, _ptr(buf), buf.shape[0] if buf is not None else 0),
               "llmcad_set_gemm_trace")

    def set_kernel_timing(self, on: bool):
        _check(lib().llmcad_set_kernel_timing(self.ctx, 1 if on else 0), "llmcad_set_kernel_timing")

    def get_kernel_timing(self, kind: int):
        ms, cnt = C.c_double(), C.c_int64()
        _check(lib().llmcad_get_kernel_timing(self.ctx, kind, C.byref(ms), C.byref(cnt)), "llmcad_get_kernel_timing")
        return ms.value, cnt.value

    def launch_count(self) -> int:
        return lib().llmcad_launch_count(self.ctx)

    def set_wait_limit_ns(self, ns: int):
        """Bound of every device-side wait of this context's kernels (0 = the default of 2 s)."""
        _check(lib().llmcad_set_wait_limit_ns(self.ctx, int(ns)), "llmcad_set_wait_limit_ns")

    def selftest_wait_timeout(self) -> int:
        """Runs a small GEMM chain whose grid barrier cannot complete; returns the device status word."""
        code = lib().llmcad_selftest_wait_timeout(self.ctx, _stream())
        if code < 0:
            raise LlmcadError(code, "llmcad_selftest_wait_timeout")
        return code


def probe_bulk_copy(src: torch.Tensor, copy_bytes: int, in_flight: int):
    """(GB/s, mean latency in us) of cp.async.bulk copies streaming `src` from device memory once (llmcad_profile.h)."""
    gbs, lat = C.c_double(0.0), C.c_double(0.0)
    _check(lib().llmcad_probe_bulk_copy(_ptr(src), src.numel() * src.element_size(), int(copy_bytes), int(in_flight),
                                        _stream(), C.byref(gbs), C.byref(lat)), "llmcad_probe_bulk_copy")
    return gbs.value, lat.value


def probe_mma_sync(warps: int, accumulators: int):
    """(multiply-adds per clock and SM, SM cycles per MMA of one warp) of mma.sync.m16n8k16 bf16 (llmcad_profile.h)."""
    rate, cyc = C.c_double(0.0), C.c_double(0.0)
    _check(lib().llmcad_probe_mma_sync(int(warps), int(accumulators), _stream(), C.byref(rate), C.byref(cyc)), "llmcad_probe_mma_sync")
    return rate.value, cyc.value


def tree_attention_noalloc(q, k, v, prefix_len: int, parent, o, status=None):
    """Context-free tree attention on caller-provided buffers (the library allocates nothing):
    q, o [n][H][128] bf16; k, v [H][kv_stride][128] bf16; parent int32[n]; status int32[1] or None."""
    n, H = q.shape[0], q.shape[1]
    # the entry point takes raw pointers: what it cannot see (dtype, shapes) is checked here
    for name, t in (("q", q), ("k", k), ("v", v), ("o", o)):
        if t.dtype != torch.bfloat16 or t.dim() != 3 or t.shape[2] != 128:
            raise ValueError(f"{name} must be a bf16 tensor [..][..][128], got {t.dtype} {tuple(t.shape)}")
    if k.shape != v.shape or k.shape[0] != H or o.shape != q.shape:
        raise ValueError("shapes: q, o [n][H][128]; k, v [H][kv_stride][128]")
    if parent.dtype != torch.int32 or parent.numel() != n or (status is not None and status.dtype != torch.int32):
        raise ValueError("parent must be int32[n] and status int32[1]")
    code = lib().llmcad_tree_attention_noalloc(_ptr(q), _ptr(k), _ptr(v), H, k.shape[1], prefix_len, _ptr(parent), n, _ptr(o),
                                               _ptr(status), _stream())
    if code != OK:
        raise LlmcadError(code, "llmcad_tree_attention_noalloc: " + lib().llmcad_noalloc_last_error().decode())
    return o


def quantize_int4(w: torch.Tensor):
    """INT4 codes [n_out][n_in] and group exponents [n_out][n_in / 64] (both int8, on w's device) of a bf16 matrix."""
    n_out, n_in = w.shape
    q = torch.empty((n_out, n_in), dtype=torch.int8, device=w.device)
    e = torch.empty((n_out, n_in // 64), dtype=torch.int8, device=w.device)
    _check(lib().llmcad_quantize_int4(_ptr(w), n_out, n_in, _ptr(q), _ptr(e), _stream()), "llmcad_quantize_int4")
    return q, e


def tree_confidence(branch_conf) -> float:
    """T_c of Sec. 3.3: the largest cumulative branch confidence (host arithmetic)."""
    c = (C.c_double * len(branch_conf))(*[float(x) for x in branch_conf])
    out = C.c_double(0.0)
    f = lib().llmcad_tree_confidence
    f.argtypes = [C.POINTER(C.c_double), C.c_int32, C.POINTER(C.c_double)]
    _check(f(c, len(branch_conf), C.byref(out)), "llmcad_tree_confidence")
    return out.value


def update_threshold(alpha: float, n_correct: int, n_all: int, t_c: float) -> float:
    """Eq. 3: the self-adaptive fallback threshold after one verification (host arithmetic)."""
    out = C.c_double(0.0)
    f = lib().llmcad_update_threshold
    f.argtypes = [C.c_double, C.c_int32, C.c_int32, C.c_double, C.POINTER(C.c_double)]
    _check(f(alpha, n_correct, n_all, t_c, C.byref(out)), "llmcad_update_threshold")
    return out.value


def tree_branches(parent_idx, node_conf):
    """Branches (root-to-leaf paths) of a token tree: (leaf ids, cumulative confidences, draft tokens per
    branch), Sec. 3.2 (host arithmetic)."""
    n = len(parent_idx)
    par = (C.c_int32 * n)(*[int(x) for x in parent_idx])
    conf = (C.c_double * n)(*[float(x) for x in node_conf])
    leaf = (C.c_int32 * n)()
    cum = (C.c_double * n)()
    length = (C.c_int32 * n)()
    nb = C.c_int32(0)
    f = lib().llmcad_tree_branches
    f.argtypes = [C.POINTER(C.c_int32), C.POINTER(C.c_double), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_double),
                  C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    _check(f(par, conf, n, leaf, cum, length, C.byref(nb)), "llmcad_tree_branches")
    return list(leaf[:nb.value]), list(cum[:nb.value]), list(length[:nb.value])


def branch_pacer(cum_conf, branch_len, m_tokens: float):
    """Eq. 1-2: (f(x) per branch, index of the branch that gets the next token) (host arithmetic)."""
    n = len(cum_conf)
    c = (C.c_double * n)(*[float(x) for x in cum_conf])
    t = (C.c_int32 * n)(*[int(x) for x in branch_len])
    out = (C.c_double * n)()
    nxt = C.c_int32(-1)
    f = lib().llmcad_branch_pacer
    f.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_int32), C.c_int32, C.c_double, C.POINTER(C.c_double),
                  C.POINTER(C.c_int32)]
    _check(f(c, t, n, float(m_tokens), out, C.byref(nxt)), "llmcad_branch_pacer")
    return list(out), nxt.value


def tree_prep(parent: torch.Tensor, prefix_len: int):
    n = parent.numel()
    dev = parent.device
    depth = torch.empty(n, dtype=torch.int32, device=dev)
    pos = torch.empty(n, dtype=torch.int32, device=dev)
    anc = torch.empty((n, 4), dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    _check(lib().llmcad_tree_prep(_ptr(parent), n, prefix_len, _ptr(depth), _ptr(pos), _ptr(anc), _ptr(status), _stream()),
           "llmcad_tree_prep")
    return depth, pos, anc, status


def anc_to_bool(anc: np.ndarray, n: int) -> np.ndarray:
    """Unpack [n][4] 32-bit words into an [n][n] 0/1 matrix (test helper)."""
    a = anc.astype(np.uint32)
    out = np.zeros((n, n), np.uint8)
    for j in range(n):
        out[:, j] = (a[:, j >> 5] >> np.uint32(j & 31)) & 1
    return out
