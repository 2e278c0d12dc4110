"""One sparsification pass of the paper's Algorithm 1 over a set of coupled pair groups, on the GPU.

Control flow and buffer plumbing only: every arithmetic step is a call into libecospa
(importance and scores -> choice of the least important pairs -> cumulative-threshold counts and
aligned selection -> physical removal from the weights, their gradients and any further tensor over
the same shared axis, e.g. optimizer moments and biases).  The kept counts are data dependent, so
the pass reads them back once before it sizes the compacted tensors; after a pass the pairs of a
group (heads) generally have different widths, which the next pass handles by describing every
pair on its own.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch

from . import binding as B
from .block import alloc_compacted


@dataclass
class Group:
    """Tensors that share one shared axis of total extent sum(widths); pair s owns widths[s] consecutive indices."""
    w1: torch.Tensor
    w2: torch.Tensor
    layout1: int
    layout2: int
    widths: List[int]
    w1b: Optional[torch.Tensor] = None                       # SwiGLU: w1 = gate, w1b = up
    g1: Optional[torch.Tensor] = None                        # gradients of w1, w2 (, w1b): needed for the importance
    g2: Optional[torch.Tensor] = None
    g1b: Optional[torch.Tensor] = None
    aux: List[Tuple[torch.Tensor, int]] = field(default_factory=list)   # (tensor, layout): moments, biases (1-D)
    rope: int = B.ROPE_NONE                                  # Q/K groups under rotary embedding: rotation pairs leave whole

    @property
    def D(self) -> int:
        return sum(self.widths)

    def n_params(self) -> int:
        other1 = self.w1.shape[0] if self.layout1 == B.SHARED_COLS else self.w1.shape[1]
        other2 = self.w2.shape[0] if self.layout2 == B.SHARED_COLS else self.w2.shape[1]
        return self.D * (other1 * (2 if self.w1b is not None else 1) + other2)


def _slice(t: Optional[torch.Tensor], layout: int, off: int, width: int) -> Optional[torch.Tensor]:
    if t is None:
        return None
    if t.dim() == 1:
        return t[off:off + width]
    return t[:, off:off + width] if layout == B.SHARED_COLS else t[off:off + width, :]


def _trim(t: Optional[torch.Tensor], layout: int, D: int) -> Optional[torch.Tensor]:
    """Drops the pad columns of a compacted buffer (a view; the pitch stays)."""
    if t is None:
        return None
    if t.dim() == 1:
        return t[:D]
    return t[:, :D] if layout == B.SHARED_COLS else t[:D, :]


def describe(groups: Sequence[Group]):
    """Pair descriptors of all groups for the scoring call, with where each described pair sits.

    A group whose pairs all have the same width is one descriptor (n_seg pairs side by side); a ragged group is
    one descriptor per pair, built on views of its tensors.  Returns (pairs, n_seg, seg_len, where, rope) with
    where[i] = (group index, offset of descriptor i inside the group's shared axis)."""
    pairs, n_seg, seg_len, where, rope = [], [], [], [], []
    for gi, g in enumerate(groups):
        kind = B.PAIR_SWIGLU if g.w1b is not None else B.PAIR_PLAIN
        D = g.D
        t = {nm: _trim(getattr(g, nm), g.layout1 if nm in ("w1", "w1b", "g1", "g1b") else g.layout2, D)
             for nm in ("w1", "w1b", "w2", "g1", "g1b", "g2")}
        if len(set(g.widths)) == 1:
            spans = [(0, D, len(g.widths), g.widths[0])]
        else:
            spans, off = [], 0
            for wd in g.widths:
                spans.append((off, wd, 1, wd))
                off += wd
        for off, ext, ns, sl in spans:
            if sl == 0:
                continue                                   # a pair that has lost every index takes no part any more
            v = {nm: _slice(t[nm], g.layout1 if nm in ("w1", "w1b", "g1", "g1b") else g.layout2, off, ext) for nm in t}
            pairs.append(B.pair(kind, ns, sl, v["w1"], v["w2"], g.layout1, g.layout2, w1b=v["w1b"],
                                g1=v["g1"], g2=v["g2"], g1b=v["g1b"], rope=g.rope))
            n_seg.append(ns); seg_len.append(sl); where.append((gi, off)); rope.append(g.rope)
    return pairs, n_seg, seg_len, where, rope


def _c_group(g: Group, with_grads: bool = True) -> "B.Group":
    D = g.D
    t = lambda nm, lay: _trim(getattr(g, nm), lay, D)
    return B.group(t("w1", g.layout1), t("w2", g.layout2), g.layout1, g.layout2, g.widths, w1b=t("w1b", g.layout1),
                   g1=t("g1", g.layout1) if with_grads else None, g2=t("g2", g.layout2) if with_grads else None,
                   g1b=t("g1b", g.layout1) if with_grads else None, aux=[(_trim(a, lay, D), lay) for a, lay in g.aux],
                   rope=g.rope)


def step(groups: Sequence[Group], n_samples: float, top_k_ratio: float, theta: float, l1: bool = True,
         k_min: int = 1, stream=None, in_place: bool = False):
    """One pass of Algorithm 1's body: importance of every pair, the top-K share of the least important pairs,
    their scores, removal of the lowest-scored aligned indices while the remaining score mass exceeds theta, and
    the physical removal from every tensor of the group.  Returns (new groups, info).
    The pass itself is two library calls (ecospa_alg1_plan, which reads the data-dependent kept counts back, and
    ecospa_alg1_apply); this function describes the groups, allocates the compacted tensors in between and wraps
    what the workspace holds afterwards.
    in_place: the tensors shrink inside their own storage (no second copy of the model and its optimizer state):
    the new groups hold the same buffers, whose leading columns / rows are the kept part."""
    assert k_min >= 1
    dev = groups[0].w1.device
    cg = [_c_group(g) for g in groups]
    ws = torch.empty(max(16, B.ecospa_alg1_workspace_bytes(cg)), dtype=torch.uint8, device=dev)
    live = sum(1 for g in groups for w in g.widths if w > 0)
    m = min(live, int(top_k_ratio * live + 0.5))
    k = B.ecospa_alg1_plan(cg, float(n_samples), m, theta, l1, k_min, ws, stream=stream)
    new_widths, pos = [], 0
    for g in groups:
        new_widths.append(k[pos:pos + len(g.widths)])
        pos += len(g.widths)
    out_groups = []
    for g, nw in zip(groups, new_widths):
        n_kept, D = sum(nw), g.D

        def shrink(t, layout):
            if t is None:
                return None
            return t if in_place else alloc_compacted(_trim(t, layout, D), layout, n_kept)
        out_groups.append(Group(shrink(g.w1, g.layout1), shrink(g.w2, g.layout2), g.layout1, g.layout2, list(nw),
                                w1b=shrink(g.w1b, g.layout1), g1=shrink(g.g1, g.layout1), g2=shrink(g.g2, g.layout2),
                                g1b=shrink(g.g1b, g.layout1), aux=[(shrink(t, lay), lay) for t, lay in g.aux], rope=g.rope))
    if in_place:
        B.ecospa_alg1_apply(cg, k, None, ws, in_place=True, stream=stream)
    else:
        # the output descriptors carry the buffers as allocated (padded pitch); their widths are not read
        og = []
        for g, ng in zip(groups, out_groups):
            og.append(B.group(ng.w1, ng.w2, g.layout1, g.layout2, ng.widths, w1b=ng.w1b, g1=ng.g1, g2=ng.g2, g1b=ng.g1b,
                              aux=ng.aux, rope=g.rope))
        B.ecospa_alg1_apply(cg, k, og, ws, in_place=False, stream=stream)
    o_ups, o_fis, o_chosen, o_kept, total_d, total_pairs = B.ecospa_alg1_offsets(cg)
    f32v = lambda off, n: ws[off:off + 4 * n].view(torch.float32)
    i32v = lambda off, n: ws[off:off + 4 * n].view(torch.int32)
    kept_lists, ko = [], 0
    for nw in new_widths:
        kept_lists.append(i32v(o_kept + 4 * ko, sum(nw)))
        ko += sum(nw)
    info = {"k": [list(nw) for nw in new_widths], "kept": kept_lists, "fisher": f32v(o_fis, total_pairs),
            "chosen": i32v(o_chosen, total_pairs), "upsilon": f32v(o_ups, total_d), "n_chosen": m, "workspace": ws}
    return out_groups, info


def total_params(groups: Sequence[Group]) -> int:
    """Param(W_t) of Algorithm 1 restricted to the coupled pairs: elements of every W_1 (gate and up) and W_2."""
    return sum(g.n_params() for g in groups)


def run_to_budget(groups: Sequence[Group], budget: int, n_samples: float, top_k_ratio: float, theta: float,
                  l1: bool = True, k_min: int = 1, refresh=None, max_passes: int = 1000, stream=None,
                  in_place: bool = False):
    """Algorithm 1's outer rule: while the model is larger than the target size c (`budget`, in parameters of the
    coupled pairs), run one pass of the body.  `refresh(groups, t)` stands for the optimizer update between two
    passes (it may overwrite the weights and gradients of the groups in place); without it the compacted gradients
    of the previous pass are reused.  Stops early when a pass removes nothing (every chosen pair is at k_min or
    within theta).  Returns (groups, history) with one entry per pass: parameters before / after and the pass info."""
    history = []
    t = 0
    while total_params(groups) > budget and t < max_passes:
        if refresh is not None:
            refresh(groups, t)
        before = total_params(groups)
        groups, info = step(groups, n_samples, top_k_ratio, theta, l1=l1, k_min=k_min, stream=stream, in_place=in_place)
        after = total_params(groups)
        history.append({"pass": t, "params_before": before, "params_after": after, "info": info})
        t += 1
        if after == before:
            break
    return groups, history
