"""Seeded synthetic workloads: shapes, value distributions and kept counts.

This module only *draws inputs*.  It holds none of the method's arithmetic
(no scores, no selection, no layer math), so both the CPU oracle's tests and
the CUDA path's tests/benchmarks can take their tensors from here without
sharing any computation.

Shapes follow the transformer notation of Eq. 1-3: d_m model width, h heads of
width d_h (d_m = h * d_h), FFN hidden width d; T = batch * seq tokens.
Storage orientation is the one the equations are written in:

* W_Q, W_K, W_V : d_m x (h*d_h) row-major, head i in columns [i*d_h,(i+1)*d_h)
  -> the shared (removable) index is the fast axis ("shared cols").
* W_O           : (h*d_h) x d_m row-major, head i is row block i (Eq. 5)
  -> the shared index is the slow axis ("shared rows").
* W_in / W_gate / W_up : d_m x d  (shared cols);  W_out / W_down : d x d_m
  (shared rows).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import torch

SHARED_COLS = 0
SHARED_ROWS = 1


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    d_m: int
    n_heads: int
    d_h: int
    d_ffn: int
    ffn: str            # "gelu" | "swiglu"
    dtype: str          # "f32" | "bf16"
    batch: int
    seq: int
    w_std: float
    g_std: float
    bias: bool
    heavy_tail: bool = False
    seed: int = 0

    @property
    def tokens(self) -> int:
        return self.batch * self.seq

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


WORKLOADS: Dict[str, Workload] = {
    # one block, fp32; the small case an oracle finishes in seconds
    "block_f32": Workload("block_f32", 1, 256, 4, 64, 1024, "gelu", "f32", 4, 128, 0.02, 0.02, True),
    # GPT-2-Medium shape
    "gpt2m": Workload("gpt2m", 24, 1024, 16, 64, 4096, "gelu", "bf16", 8, 1024, 0.02, 1e-3, True),
    # LLaMA-1B shape
    "llama1b": Workload("llama1b", 22, 2048, 32, 64, 5632, "swiglu", "bf16", 4, 2048, 0.02, 1e-3, False),
    # LLaMA-7B single layer, heavy-tailed importance
    "llama7b_layer": Workload("llama7b_layer", 1, 4096, 32, 128, 11008, "swiglu", "bf16", 2, 4096, 0.02, 1e-3,
                              False, heavy_tail=True),
    # tail-shape case: d_m = 768, 12 heads x 64, FFN 3072 (GPT-2-Small shape, Table "gpt2_dims")
    "tails768": Workload("tails768", 1, 768, 12, 64, 3072, "gelu", "bf16", 2, 160, 0.02, 1e-3, True),
    # tiny SwiGLU block for fast CPU tests
    "tiny_swiglu": Workload("tiny_swiglu", 1, 64, 2, 32, 160, "swiglu", "bf16", 2, 24, 0.02, 1e-3, False),
}

# kept counts that the paper's own compressed models show (Tables "deit_dims"/"gpt2_dims"):
RAGGED_HEAD_KEPT = [20, 21, 25, 26, 30, 37, 64]
RAGGED_FFN_KEPT = [1073, 1337, 2044]


def kept_count(seg_len: int, sparsity: float) -> int:
    """k = round((1 - s) * seg_len), half away from zero, at least 1."""
    k = int(math.floor((1.0 - sparsity) * seg_len + 0.5))
    return max(1, min(seg_len, k))


_TENSOR_KINDS = ["wq", "wk", "wv", "wo", "w1", "w1b", "w2", "b1", "b2", "bq", "bk", "bv",
                 "gq", "gk", "gv", "go", "g1", "g1b", "g2",
                 "x", "dq", "dk", "dv", "dout", "dy", "ctx",
                 "tail_wq", "tail_wk", "tail_wv", "tail_wo", "tail_w1", "tail_w1b", "tail_w2",
                 "m1", "v1"]


def tensor_seed(seed: int, layer: int, kind: str, step: int = 0) -> int:
    """One integer seed per (workload seed, layer, tensor kind, re-draw step)."""
    kid = _TENSOR_KINDS.index(kind)
    return ((seed * 1_000_003 + layer) * 1009 + kid) * 131 + step + 12345


def _randn(shape, std: float, dtype: torch.dtype, seed: int, device: str) -> torch.Tensor:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    t = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        t.mul_(std)
    return t.to(dtype)


def _heavy_tail_(t: torch.Tensor, shared_axis: int, seed: int, frac: float = 0.05, scale: float = 10.0) -> None:
    """Scale a seeded `frac` subset of the shared-index vectors of `t` by `scale` (in place)."""
    n = t.shape[shared_axis]
    g = torch.Generator(device="cpu")
    g.manual_seed(seed ^ 0x5EED)
    idx = torch.randperm(n, generator=g)[: max(1, int(round(frac * n)))].to(t.device)
    if shared_axis == 1:
        t[:, idx] = (t[:, idx].float() * scale).to(t.dtype)
    else:
        t[idx, :] = (t[idx, :].float() * scale).to(t.dtype)


def layer_weights(w: Workload, layer: int, device: str = "cpu") -> Dict[str, torch.Tensor]:
    """Weights (and biases) of one block in the orientation described in the module docstring."""
    dt = w.torch_dtype
    D = w.n_heads * w.d_h
    out: Dict[str, torch.Tensor] = {}
    for kind in ("wq", "wk", "wv"):
        out[kind] = _randn((w.d_m, D), w.w_std, dt, tensor_seed(w.seed, layer, kind), device)
    out["wo"] = _randn((D, w.d_m), w.w_std, dt, tensor_seed(w.seed, layer, "wo"), device)
    out["w1"] = _randn((w.d_m, w.d_ffn), w.w_std, dt, tensor_seed(w.seed, layer, "w1"), device)
    if w.ffn == "swiglu":
        out["w1b"] = _randn((w.d_m, w.d_ffn), w.w_std, dt, tensor_seed(w.seed, layer, "w1b"), device)
    out["w2"] = _randn((w.d_ffn, w.d_m), w.w_std, dt, tensor_seed(w.seed, layer, "w2"), device)
    if w.bias:
        out["b1"] = _randn((w.d_ffn,), w.w_std, dt, tensor_seed(w.seed, layer, "b1"), device)
        out["b2"] = _randn((w.d_m,), w.w_std, dt, tensor_seed(w.seed, layer, "b2"), device)
        for kind in ("bq", "bk", "bv"):
            out[kind] = _randn((D,), w.w_std, dt, tensor_seed(w.seed, layer, kind), device)
    if w.heavy_tail:
        for kind in ("wq", "wk", "wv", "w1", "w1b"):
            if kind in out:
                _heavy_tail_(out[kind], 1, tensor_seed(w.seed, layer, "tail_" + kind))
        for kind in ("wo", "w2"):
            _heavy_tail_(out[kind], 0, tensor_seed(w.seed, layer, "tail_" + kind))
    return out


_GRAD_OF = {"gq": "wq", "gk": "wk", "gv": "wv", "go": "wo", "g1": "w1", "g1b": "w1b", "g2": "w2"}


def layer_grads(w: Workload, layer: int, step: int = 0, device: str = "cpu") -> Dict[str, torch.Tensor]:
    """Weight gradients of one block: same shapes/dtype as the weights, N(0, g_std^2); `step` re-draws."""
    dt = w.torch_dtype
    D = w.n_heads * w.d_h
    shapes = {"gq": (w.d_m, D), "gk": (w.d_m, D), "gv": (w.d_m, D), "go": (D, w.d_m),
              "g1": (w.d_m, w.d_ffn), "g1b": (w.d_m, w.d_ffn), "g2": (w.d_ffn, w.d_m)}
    out = {}
    for kind, shp in shapes.items():
        if kind == "g1b" and w.ffn != "swiglu":
            continue
        out[kind] = _randn(shp, w.g_std, dt, tensor_seed(w.seed, layer, kind, step), device)
    return out


def activations(w: Workload, layer: int, tokens: Optional[int] = None, device: str = "cpu",
                kinds: Optional[List[str]] = None, widths: Optional[Dict[str, int]] = None) -> Dict[str, torch.Tensor]:
    """N(0,1) activations and upstream gradients.  `widths` gives the column count of
    tensors whose width depends on the kept counts (dq, dk, dv, ctx); others are d_m wide."""
    dt = w.torch_dtype
    T = tokens if tokens is not None else w.tokens
    kinds = kinds or ["x", "dy", "dout"]
    widths = widths or {}
    out = {}
    for kind in kinds:
        ncol = widths.get(kind, w.d_m)
        out[kind] = _randn((T, ncol), 1.0, dt, tensor_seed(w.seed, layer, kind), device)
    return out


def kept_plan(w: Workload, sparsity: float) -> Dict[str, List[int]]:
    """Per-segment kept counts for the three pair groups of a block at one sparsity."""
    kh = kept_count(w.d_h, sparsity)
    return {"qk": [kh] * w.n_heads, "vo": [kh] * w.n_heads, "ffn": [kept_count(w.d_ffn, sparsity)]}


def model_bytes(w: Workload) -> int:
    """Bytes of all coupled-pair weight matrices of the model (no biases)."""
    D = w.n_heads * w.d_h
    per_layer = 4 * w.d_m * D + (3 if w.ffn == "swiglu" else 2) * w.d_m * w.d_ffn
    return per_layer * w.n_layers * w.elem_bytes
