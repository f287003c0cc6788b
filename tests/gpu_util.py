"""Helpers shared by the GPU parity tests: build a verifier and its oracle twin from the
same seeded bytes, run both, compare."""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional

import numpy as np
import torch

from oracle import oracle as orc
from paper_2309_04255_b200 import binding as B
from paper_2309_04255_b200 import inputs as gen

F32_TOL = 1e-4    # fp32 logits: max|delta| <= 1e-4 * max|logit|
BF16_TOL = 2e-2   # bf16 logits: max|delta| <= 2e-2 * max|logit|


class Twin:
    """A model instantiated on both sides. Weights are generated layer by layer on the host,
    uploaded and packed; the oracle keeps (or regenerates) the same host tensors."""

    def __init__(self, cfg, max_seq: int, flags: int = 0, seed: int = 0, keep_host: bool = True, scale: float = 1.0):
        self.cfg, self.seed, self.scale = cfg, seed, scale
        self.v = B.Verifier(cfg, max_seq, flags=flags)
        self.keep_host = keep_host
        self.layers: Dict[int, Dict[str, torch.Tensor]] = {}
        self.glob = self._scaled(gen.gen_globals(cfg, seed))
        self.v.pack_globals(self.glob)
        with ThreadPoolExecutor(4) as ex:
            for l, w in enumerate(ex.map(lambda l: self._scaled(gen.gen_layer(cfg, l, seed)), range(cfg.n_layers))):
                self.v.pack_layer(l, w)
                if keep_host:
                    self.layers[l] = w

    def _scaled(self, w):
        if self.scale == 1.0:
            return w
        return {k: (v if k.endswith("norm") else (v.float() * self.scale).to(v.dtype)) for k, v in w.items()}

    def layer(self, l: int):
        if l in self.layers:
            return self.layers[l]
        return self._scaled(gen.gen_layer(self.cfg, l, self.seed))

    # ---- synthetic prefix cache: same values on both sides
    def fill_prefix_synthetic(self, P: int):
        kvv = self.v.kv_view()
        self._prefix = {}
        for l in range(self.cfg.n_layers):
            k, v = gen.gen_prefix_kv(self.cfg, l, P, self.seed)
            kvv[l, 0, :, :P] = k.to(kvv.device)
            kvv[l, 1, :, :P] = v.to(kvv.device)
            self._prefix[l] = (k, v)

    def prefix_fn(self, l: int):
        return self._prefix[l]

    def oracle_pass(self, P: int, tokens, parent, prefix_fn=None):
        return orc.verify_tree(self.cfg, self.glob, self.layer, prefix_fn or self.prefix_fn, P, tokens, parent)

    def gpu_pass(self, P: int, tokens, parent, want_logits=True):
        dev = self.v.device
        t = torch.as_tensor(np.asarray(tokens, np.int32), device=dev)
        p = torch.as_tensor(np.asarray(parent, np.int32), device=dev)
        out = self.v.verify_tree(P, t, p, want_logits=want_logits)
        torch.cuda.synchronize()
        return {k: (v.cpu().numpy() if v is not None else None) for k, v in out.items()}


def logits_close(gpu: np.ndarray, ref: np.ndarray, tol: float):
    scale = np.abs(ref).max()
    err = np.abs(gpu.astype(np.float64) - ref).max()
    assert np.isfinite(gpu).all()
    assert err <= tol * scale, f"max|delta| {err:.3e} > {tol} * max|logit| {scale:.3e}"
    return err / scale


def argmax_agrees_where_decided(gpu_argmax, ref_logits, tol: float):
    """Wherever the oracle's top-2 margin exceeds the logit tolerance the argmax must agree."""
    scale = np.abs(ref_logits).max()
    srt = np.sort(ref_logits, axis=1)
    margin = srt[:, -1] - srt[:, -2]
    decided = margin > tol * scale
    ref_arg = ref_logits.argmax(1)
    assert (gpu_argmax[decided] == ref_arg[decided]).all()
    return int((~decided).sum())


def check_acceptance_against_oracle(out, tokens, parent):
    """The oracle's search run on the GPU's own argmax must give the GPU's path, bit for bit."""
    n = len(tokens)
    acc = orc.accept(parent, tokens, out["argmax"][:n])
    s = out["scalars"]
    assert s[B.S_STATUS] == 0
    assert s[B.S_ACCEPTED_LEN] == acc.accepted_len
    assert out["accepted_path"][: acc.accepted_len].tolist() == acc.path.tolist()
    assert s[B.S_NEXT_TOKEN] == acc.next_token
    assert s[B.S_N_CORRECT] == acc.n_correct and s[B.S_N_ALL] == acc.n_all and s[B.S_RECTIFIED] == acc.rectified
    return acc


def cache_rows(v: B.Verifier, upto: int) -> np.ndarray:
    """[L][2][H][upto][hd] as float64."""
    return v.kv_view()[:, :, :, :upto].double().cpu().numpy()
