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


def step(groups: Sequence[Group], n_samples: float, top_k_ratio: float, theta: float, l1: bool = True,
         k_min: int = 1, stream=None, in_place: bool = False):
    """One pass of Algorithm 1's body: importance of every pair, the top-K share of the least important pairs,
    their scores, removal of the lowest-scored aligned indices while the remaining score mass exceeds theta, and
    the physical removal from every tensor of the group.  Returns (new groups, info).
    in_place: the tensors shrink inside their own storage (no second copy of the model and its optimizer state):
    the new groups hold the same buffers, whose leading columns / rows are the kept part."""
    assert k_min >= 1 and all(w >= 1 for g in groups for w in g.widths)
    dev = groups[0].w1.device
    pairs, n_seg, seg_len, where, rope = describe(groups)
    total_segs = sum(n_seg)
    total_d = sum(a * b for a, b in zip(n_seg, seg_len))
    i32, f32 = torch.int32, torch.float32
    ups = torch.empty(total_d, dtype=f32, device=dev)
    fis = torch.empty(total_segs, dtype=f32, device=dev)
    ws = torch.empty(max(16, B.ecospa_score_workspace_bytes(pairs)), dtype=torch.uint8, device=dev)
    B.ecospa_score_pairs(pairs, float(n_samples), ups, None, fis, ws, stream=stream)
    m = min(total_segs, int(top_k_ratio * total_segs + 0.5))
    chosen = torch.empty(total_segs, dtype=i32, device=dev)
    B.ecospa_choose_pairs(fis, m, chosen, stream=stream)
    slots = torch.empty(total_d, dtype=i32, device=dev)
    k_out = torch.empty(total_segs, dtype=i32, device=dev)
    B.ecospa_select_aligned_threshold(ups, n_seg, seg_len, theta, slots, k_out, l1=l1, k_min=k_min, chosen=chosen,
                                      rope=rope if any(rope) else None, stream=stream)
    k = k_out.cpu().tolist()                 # the one read-back: the counts size everything that follows

    # per group: the kept list of the whole shared axis, then one gather per tensor
    new_widths: List[List[int]] = [[] for _ in groups]
    src: List[List[int]] = [[] for _ in groups]
    add: List[List[int]] = [[] for _ in groups]
    kk: List[List[int]] = [[] for _ in groups]
    seg, d_off = 0, 0
    for (gi, off), ns, sl in zip(where, n_seg, seg_len):
        for s in range(ns):
            new_widths[gi].append(k[seg]); kk[gi].append(k[seg])
            src[gi].append(d_off + s * sl); add[gi].append(off)      # slot indices are relative to the described pair group
            seg += 1
        d_off += ns * sl
    out_groups, kept_lists, jobs = [], [], []
    for gi, g in enumerate(groups):
        n_kept = sum(kk[gi])
        dst, run = [], 0
        for v in kk[gi]:
            dst.append(run); run += v
        kept = torch.empty(max(n_kept, 1), dtype=i32, device=dev)
        B.ecospa_pack_kept(slots, src[gi], dst, kk[gi], add[gi], kept, stream=stream)
        kept_lists.append(kept[:n_kept])
        D = g.D

        def shrink(t, layout):
            if t is None:
                return None
            if in_place:
                v = _trim(t, layout, D)
                jobs.append(B.gather(v, v, layout, kept, n_kept, D))
                return t                                   # same storage and pitch; `widths` says what is valid
            o = alloc_compacted(_trim(t, layout, D), layout, n_kept)
            jobs.append(B.gather(_trim(t, layout, D), o, layout, kept, n_kept, D))
            return o
        ng = Group(shrink(g.w1, g.layout1), shrink(g.w2, g.layout2), g.layout1, g.layout2, new_widths[gi],
                   w1b=shrink(g.w1b, g.layout1), g1=shrink(g.g1, g.layout1), g2=shrink(g.g2, g.layout2),
                   g1b=shrink(g.g1b, g.layout1), aux=[(shrink(t, lay), lay) for t, lay in g.aux], rope=g.rope)
        out_groups.append(ng)
    (B.ecospa_compact_tensors_inplace if in_place else B.ecospa_compact_tensors)(jobs, stream=stream)
    info = {"k": new_widths, "kept": kept_lists, "fisher": fis, "chosen": chosen, "upsilon": ups, "n_chosen": m}
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
