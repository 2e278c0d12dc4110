"""Descriptor plumbing for whole transformer blocks: which stored tensors form which coupled pairs.

No arithmetic here: this module only names the three pair groups of a block (Eq. 5 and the FFN
pair of Sec. 3.1) in terms of the stored tensors, allocates outputs, and calls the binding.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import torch

from . import binding as B

GROUPS = ("qk", "vo", "ffn")


def block_pairs(w: Dict[str, torch.Tensor], n_heads: int, d_h: int, d_ffn: int,
                g: Optional[Dict[str, torch.Tensor]] = None, layout_in: int = B.SHARED_COLS,
                layout_out: int = B.SHARED_ROWS) -> List[B.Pair]:
    """[QK, VO, FFN] pair groups of one block.

    QK: column j of head i of W^Q with column j of head i of W^K (W_1 = W_i^Q, W_2 = W_i^K^T).
    VO: column j of head i of W^V with row j of row-block i of W^O.
    FFN: column j of W_in (or of W_gate (.) W_up) with row j of W_out (W_down).
    layout_in: storage of W^Q, W^K, W^V, W_in / W_gate / W_up (default: as the equations write them, d_m x D);
    layout_out: storage of W^O, W_out / W_down (default D x d_m).
    """
    g = g or {}
    swiglu = "w1b" in w
    return [
        B.pair(B.PAIR_PLAIN, n_heads, d_h, w["wq"], w["wk"], layout_in, layout_in,
               g1=g.get("gq"), g2=g.get("gk")),
        B.pair(B.PAIR_PLAIN, n_heads, d_h, w["wv"], w["wo"], layout_in, layout_out,
               g1=g.get("gv"), g2=g.get("go")),
        B.pair(B.PAIR_SWIGLU if swiglu else B.PAIR_PLAIN, 1, d_ffn, w["w1"], w["w2"], layout_in, layout_out,
               w1b=w.get("w1b"), g1=g.get("g1"), g2=g.get("g2"), g1b=g.get("g1b")),
    ]


def pad8(n: int, elem_bytes: int = 2) -> int:
    """Row pitch (elements) that keeps rows 16-byte aligned."""
    v = 16 // elem_bytes
    return (n + v - 1) // v * v


def alloc_compacted(t: torch.Tensor, layout: int, n_kept: int) -> torch.Tensor:
    """Output buffer for the compaction of `t`; shared-cols outputs get a 16-byte aligned pitch
    (returned tensor is the full padded buffer: shape (other, pitch))."""
    if t.dim() == 1:
        return torch.empty(pad8(n_kept, t.element_size()), dtype=t.dtype, device=t.device)
    if layout == B.SHARED_COLS:
        return torch.empty((t.shape[0], pad8(n_kept, t.element_size())), dtype=t.dtype, device=t.device)
    return torch.empty((n_kept, t.shape[1]), dtype=t.dtype, device=t.device)


def padded_head_layout(k_heads: Sequence[int], multiple: int = 16) -> Tuple[List[int], List[int], int]:
    """Column blocks of compacted heads padded to the width granularity of the attention kernels:
    (first column of every head, its padded width, total padded width)."""
    off, w, o = [], [], 0
    for k in k_heads:
        kp = (int(k) + multiple - 1) // multiple * multiple
        off.append(o); w.append(kp)
        o += kp
    return off, w, o
