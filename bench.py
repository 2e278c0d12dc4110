"""Benchmark of the coupled-sparsity hot path on a LLaMA-1B-shaped model (or another workload).

One step = one pass of the whole hot path over every layer of the model:
  score (+ Fisher) of all coupled pairs -> aligned top-k -> compaction of weights, biases and
  gradients -> forward and backward of every compacted block (Q/K/V projections, attention core on the
  compacted heads, output projection, FFN).

    python bench.py --gpus 1 --steps 10 --warmup 3
    python bench.py --impl reference            # the CPU oracle on a bounded sample of the same step

Prints one JSON line (rank 0).  `value` is the tensor-core throughput of the step (algorithmic
flops of every product of the step / whole step time); the memory-bound phase is reported
alongside as GB/s, and the projection / FFN products and the attention core are also replayed
on their own for their rooflines.  With N > 1 every rank runs an independent replica (the path has no exchange
step); times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes (read + write) per gemm_kernel launch, averaged over the eight GEMM launches of a layer:
# `dram__bytes_read.sum + dram__bytes_write.sum` of one ncu capture of this build per workload (one layer captured;
# per-launch traffic does not depend on the number of layers).  Workloads without a capture: None.
NCU_GEMM_TRAFFIC_BYTES = {"gpt2m": 45.3e6, "llama1b": 213.3e6}
# DRAM bytes per step of sumsq_kernel + gather_kernel on 8 gpt2m layers under ncu (grow in proportion to the layers)
NCU_SPARSIFY_TRAFFIC_BYTES_PER_LAYER = {"gpt2m": 889.3e6 / 8}

METRIC = "compacted-pair fwd/bwd TFLOP/s over the whole coupled-sparsity step (score+select+compact GB/s alongside)"


# ---------------------------------------------------------------------------------------------
# workload accounting: algorithmic bytes (every weight and gradient element read once for the scores, the
# gather's reads and writes) and algorithmic flops (2*M*N*K of every product with the real kept counts)
# ---------------------------------------------------------------------------------------------

def step_flops(wl, n_attn: int, k_ffn: int) -> float:
    """2*M*N*K of every compacted-pair product, forward (x1) and backward (x2), all layers."""
    T, d = wl.tokens, wl.d_m
    ffn_mats = 3 if wl.ffn == "swiglu" else 2
    fwd = 2.0 * T * d * (2 * n_attn) + 2.0 * T * d * (2 * n_attn) + 2.0 * T * d * k_ffn * ffn_mats
    return 3.0 * fwd * wl.n_layers


def attention_flops(wl, k_qk: int, k_vo: int, causal: bool) -> float:
    """Products of the attention core on the compacted heads, all layers: forward S = Q K^T and P V (2 products),
    backward S again, dP, dV, dQ, dK (5 products), 2*seq*seq*width flops each per sequence and head with the real
    kept widths; a causal mask halves the pairs."""
    pairs = wl.batch * wl.n_heads * float(wl.seq) * wl.seq * (0.5 if causal else 1.0)
    fwd = 2.0 * pairs * (k_qk + k_vo)
    bwd = 2.0 * pairs * (3 * k_qk + 2 * k_vo)
    return (fwd + bwd) * wl.n_layers


def sparsify_bytes(wl, rho: float, with_grads: bool = True, transposed: bool = False) -> float:
    """Weights (and gradients) read once for the scores; compaction reads a shared-cols tensor in
    full and a shared-rows tensor at the kept fraction, and writes the kept fraction of both.
    transposed: every matrix is stored the other way round, which swaps the two kinds."""
    D = wl.n_heads * wl.d_h
    e = wl.elem_bytes
    cols = (3 * wl.d_m * D + (2 if wl.ffn == "swiglu" else 1) * wl.d_m * wl.d_ffn) * e * wl.n_layers
    rows = (wl.d_m * D + wl.d_m * wl.d_ffn) * e * wl.n_layers
    if transposed:
        cols, rows = rows, cols
    mult = 2 if with_grads else 1
    score = (cols + rows) * mult
    compact = (cols * (1 + rho) + rows * 2 * rho) * mult
    return float(score + compact)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([f.strip() for f in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# the GPU step
# ---------------------------------------------------------------------------------------------

class Model:
    """Device-resident synthetic model plus every buffer a step writes (allocated once)."""

    def __init__(self, wl, sparsity: float, device, n_act_sets: int = 4, transposed: bool = False):
        import torch
        from paper_2511_11641_b200 import binding as B, block as BL, workloads as WL
        self.wl, self.dev, self.B, self.BL = wl, device, B, BL
        self.torch = torch
        self.w, self.g, self.pairs = [], [], []
        # transposed: every weight matrix (and its gradient) stored the other way round, i.e. W_Q, W_K, W_V, W_1
        # as D x d_m (what a framework's linear layer keeps) and W_O, W_2 as d_m x D
        self.transposed = transposed
        lin, lout = (B.SHARED_ROWS, B.SHARED_COLS) if transposed else (B.SHARED_COLS, B.SHARED_ROWS)
        self.lay = dict(w_in_layout=lin, w_out_layout=lout)
        for l in range(wl.n_layers):
            w = WL.layer_weights(wl, l, device=device)
            g = WL.layer_grads(wl, l, device=device)
            if transposed:
                w = {k_: (v.t().contiguous() if v.dim() == 2 else v) for k_, v in w.items()}
                g = {k_: (v.t().contiguous() if v.dim() == 2 else v) for k_, v in g.items()}
            self.w.append(w); self.g.append(g)
            self.pairs += BL.block_pairs(w, wl.n_heads, wl.d_h, wl.d_ffn, g, layout_in=lin, layout_out=lout)
        plan = WL.kept_plan(wl, sparsity)
        self.plan = plan
        self.n_attn, self.k_ffn = sum(plan["qk"]), plan["ffn"][0]
        # The attention kernels want every head's block of Q^c, K^c, V^c padded to a multiple of 16 columns: the kept
        # lists of the two attention groups are padded with "no index" entries (zero columns) before compaction.
        self.qk_off, self.qk_w, self.n_qk_p = BL.padded_head_layout(plan["qk"])
        self.vo_off, self.vo_w, self.n_vo_p = BL.padded_head_layout(plan["vo"])
        assert self.n_qk_p == self.n_vo_p, "the benchmark keeps the same count in the QK and VO pair of a head"
        self.n_attn_p = self.n_qk_p
        self.padded = self.n_attn_p != self.n_attn
        self.causal = True     # GPT-2- and LLaMA-shaped decoders mask keys after the query
        self.scale = 1.0 / (wl.d_h ** 0.5)
        self.k_per_seg = (plan["qk"] + plan["vo"] + plan["ffn"]) * wl.n_layers
        self.n_seg = [wl.n_heads, wl.n_heads, 1] * wl.n_layers
        self.seg_len = [wl.d_h, wl.d_h, wl.d_ffn] * wl.n_layers
        D_layer = 2 * wl.n_heads * wl.d_h + wl.d_ffn
        f32, i32 = torch.float32, torch.int32
        self.ups = torch.empty(D_layer * wl.n_layers, dtype=f32, device=device)
        self.fis = torch.empty((2 * wl.n_heads + 1) * wl.n_layers, dtype=f32, device=device)
        self.kept = torch.empty(sum(self.k_per_seg), dtype=i32, device=device)
        # padded kept lists of the attention groups, layer after layer: [QK | VO]
        self.kept_p = torch.empty(2 * self.n_attn_p * wl.n_layers, dtype=i32, device=device) if self.padded else None
        self.score_ws = torch.empty(B.ecospa_score_workspace_bytes(self.pairs), dtype=torch.uint8, device=device)
        # compaction jobs: weights, biases and gradients of every pair group
        self.c, self.jobs = [], []
        off = 0
        D_attn = wl.n_heads * wl.d_h
        groups = [(["wq", "wk", "bq", "bk"], ["gq", "gk"], self.n_attn, D_attn),
                  (["wv", "wo", "bv"], ["gv", "go"], self.n_attn, D_attn),
                  (["w1", "w1b", "w2", "b1"], ["g1", "g1b", "g2"], self.k_ffn, wl.d_ffn)]
        layout = {"wq": lin, "wk": lin, "wv": lin, "wo": lout, "w1": lin, "w1b": lin, "w2": lout, "bq": 0, "bk": 0, "bv": 0,
                  "b1": 0, "gq": lin, "gk": lin, "gv": lin, "go": lout, "g1": lin, "g1b": lin, "g2": lout}
        self.layout = layout
        self.pad_args = None
        if self.padded:
            src, dst, kk, kp = [], [], [], []
            o_src, o_dst = 0, 0
            for l in range(wl.n_layers):
                for grp, widths in (("qk", self.qk_w), ("vo", self.vo_w)):
                    for h in range(wl.n_heads):
                        src.append(o_src); dst.append(o_dst); kk.append(plan[grp][h]); kp.append(widths[h])
                        o_src += plan[grp][h]; o_dst += widths[h]
                o_src += self.k_ffn
            self.pad_args = (src, dst, kk, kp)
        for l in range(wl.n_layers):
            c = {}
            for gi, (wn, gn, nk, D) in enumerate(groups):
                kd = self.kept[off:off + nk]
                nk_out = nk
                if self.padded and gi < 2:
                    nk_out = self.n_attn_p
                    kd = self.kept_p[(2 * l + gi) * nk_out:(2 * l + gi + 1) * nk_out]
                for nm in wn + gn:
                    src = self.w[l].get(nm) if nm in self.w[l] else self.g[l].get(nm)
                    if src is None:
                        continue
                    o = BL.alloc_compacted(src, layout[nm], nk_out)
                    c[nm] = o
                    self.jobs.append(B.gather(src, o, layout[nm], kd, nk_out, D))
                off += nk
            self.c.append(c)
        # activations and upstream gradients: a small pool of distinct sets cycled over the layers
        T, d, n, k = wl.tokens, wl.d_m, self.n_attn_p, self.k_ffn
        npad = BL.pad8(n)
        dt = wl.torch_dtype
        self.acts = []
        for s in range(n_act_sets):
            self.acts.append(WL.activations(wl, s, kinds=["x", "dy", "dout", "dq", "dk", "dv", "ctx"],
                                            widths={"dq": npad, "dk": npad, "dv": npad, "ctx": npad}, device=device))
        e = lambda *shape: torch.empty(shape, dtype=dt, device=device)
        self.o = {"Q": e(T, npad), "K": e(T, npad), "V": e(T, npad), "Out": e(T, d), "dX": e(T, d), "dCtx": e(T, npad),
                  "dWq": e(n, d) if transposed else e(d, npad), "dWk": e(n, d) if transposed else e(d, npad),
                  "dWv": e(n, d) if transposed else e(d, npad), "dWo": e(d, npad) if transposed else e(n, d),
                  "dbq": e(n), "dbk": e(n), "dbv": e(n), "dbo": e(d)}
        self.o["dX"].zero_()
        # attention core: mixed values, their gradient, and the gradients it hands to the projections' backward
        self.o.update({"Ctx": e(T, npad), "dQ": e(T, npad), "dK": e(T, npad), "dV": e(T, npad)})
        self.lse = torch.empty(wl.n_heads * T, dtype=f32, device=device)
        self.heads = B.heads(self.qk_off, self.qk_w, self.vo_off, self.vo_w)
        self.attn_ws = torch.empty(B.ecospa_attn_workspace_bytes(wl.batch, wl.seq, wl.n_heads), dtype=torch.uint8, device=device)
        self.has_attention = wl.torch_dtype == torch.bfloat16 and not transposed
        from paper_2511_11641_b200 import layers as L
        self.L = L
        self.act = B.ACT_SWIGLU if wl.ffn == "swiglu" else B.ACT_GELU_ERF
        self.ffn = L.ffn_buffers(T, d, k, self.act, dt, device, transposed=transposed)
        self.proj_ws = torch.empty(B.ecospa_proj_workspace_bytes(T, d, n, B.BF16 if dt == torch.bfloat16 else B.F32) + 16,
                                   dtype=torch.uint8, device=device)

    def sparsify(self):
        B = self.B
        B.ecospa_score_pairs(self.pairs, float(self.wl.tokens), self.ups, None, self.fis, self.score_ws)
        B.ecospa_select_aligned_topk(self.ups, self.n_seg, self.seg_len, self.k_per_seg, self.kept)
        if self.padded:
            B.ecospa_pad_kept(self.kept, *self.pad_args, self.kept_p)
        B.ecospa_compact_tensors(self.jobs)

    def attention_fwd(self):
        o, wl = self.o, self.wl
        self.B.ecospa_coupled_attn_fwd(o["Q"], o["K"], o["V"], wl.batch, wl.seq, self.heads, self.scale, self.causal, o["Ctx"],
                                       self.lse)

    def attention_bwd(self):
        o, wl = self.o, self.wl
        self.B.ecospa_coupled_attn_bwd(o["Q"], o["K"], o["V"], o["Ctx"], o["dCtx"], self.lse, wl.batch, wl.seq, self.heads,
                                       self.scale, self.causal, o["dQ"], o["dK"], o["dV"], self.attn_ws)

    def block(self, l: int):
        """Forward and backward of layer l as a training step meets them: Q, K, V projections -> attention core ->
        output projection -> FFN forward and backward -> output projection backward -> attention backward ->
        backward of the three projections.  Every call consumes what the previous one produced."""
        B, o, n, k = self.B, self.o, self.n_attn_p, self.k_ffn
        bias = self.wl.bias
        c, a = self.c[l], self.acts[l % len(self.acts)]
        B.ecospa_coupled_qkv_fwd(a["x"], c["wq"], c["wk"], c["wv"], n, n, o["Q"], o["K"], o["V"], bq_c=c.get("bq"),
                                 bk_c=c.get("bk"), bv_c=c.get("bv"), workspace=self.proj_ws, **self.lay)
        self.attention_fwd()
        B.ecospa_coupled_vo_fwd_o(o["Ctx"], c["wo"], n, o["Out"], workspace=self.proj_ws, **self.lay)
        self.L.ffn_fwd_bwd(a["x"], a["dy"], self.act, c["w1"], c["w2"], k, self.ffn, w1bc=c.get("w1b"),
                           b1c=c.get("b1"), b2=self.w[l].get("b2"), bias_grads=self.wl.bias, **self.lay)
        B.ecospa_coupled_vo_bwd_o(o["Ctx"], c["wo"], n, a["dout"], o["dCtx"], o["dWo"], o["dbo"] if bias else None,
                                  workspace=self.proj_ws, **self.lay)
        self.attention_bwd()
        B.ecospa_coupled_qkv_bwd(a["x"], c["wq"], c["wk"], c["wv"], n, n, o["dQ"], o["dK"], o["dV"], o["dX"], o["dWq"],
                                 o["dWk"], o["dWv"], o["dbq"] if bias else None, o["dbk"] if bias else None,
                                 o["dbv"] if bias else None, accumulate_dX=True, workspace=self.proj_ws, **self.lay)

    def blocks(self):
        for l in range(self.wl.n_layers):
            self.block(l)

    def attention_only(self):
        """The attention calls of a step on their own (for their share of the step time)."""
        for l in range(self.wl.n_layers):
            self.attention_fwd()
            self.attention_bwd()

    def layer(self, l: int):
        """Forward and backward of the compacted QK / VO / FFN pairs of layer l (the projections and the FFN only:
        the attention-mixed values and the gradients of Q^c, K^c, V^c come from the input pool)."""
        B, o, n, k = self.B, self.o, self.n_attn_p, self.k_ffn
        bias = self.wl.bias
        c, a = self.c[l], self.acts[l % len(self.acts)]
        # forward: Q, K, V in one launch; (attention core is the caller's); output projection; FFN
        B.ecospa_coupled_qkv_fwd(a["x"], c["wq"], c["wk"], c["wv"], n, n, o["Q"], o["K"], o["V"], bq_c=c.get("bq"),
                                 bk_c=c.get("bk"), bv_c=c.get("bv"), workspace=self.proj_ws, **self.lay)
        B.ecospa_coupled_vo_fwd_o(a["ctx"], c["wo"], n, o["Out"], workspace=self.proj_ws, **self.lay)
        # FFN forward + backward
        self.L.ffn_fwd_bwd(a["x"], a["dy"], self.act, c["w1"], c["w2"], k, self.ffn, w1bc=c.get("w1b"),
                           b1c=c.get("b1"), b2=self.w[l].get("b2"), bias_grads=self.wl.bias, **self.lay)
        # backward: what dOut gives (dCtx, dW_O), then what dQ, dK, dV give (dW_Q, dW_K, dW_V, dX)
        B.ecospa_coupled_vo_bwd_o(a["ctx"], c["wo"], n, a["dout"], o["dCtx"], o["dWo"], o["dbo"] if bias else None,
                                  workspace=self.proj_ws, **self.lay)
        B.ecospa_coupled_qkv_bwd(a["x"], c["wq"], c["wk"], c["wv"], n, n, a["dq"], a["dk"], a["dv"], o["dX"], o["dWq"],
                                 o["dWk"], o["dWv"], o["dbq"] if bias else None, o["dbk"] if bias else None,
                                 o["dbv"] if bias else None, accumulate_dX=True, workspace=self.proj_ws, **self.lay)

    def layers(self):
        for l in range(self.wl.n_layers):
            self.layer(l)

    def host_copies(self):
        """Pinned host mirrors of every input of a step (weights, gradients, activations)."""
        torch = self.torch
        pairs = []
        for d in self.w + self.g + self.acts:
            for t in d.values():
                h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
                h.copy_(t)
                pairs.append((h, t))
        return pairs


def max_over_ranks(values, device=None):
    """Element-wise maximum of per-rank timings over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(world: int, units_per_rank: float, ms: float) -> float:
    """Whole-job rate: every rank processed `units_per_rank` in `ms` (already the max over ranks)."""
    return world * units_per_rank / ms


def tensor_peak(peaks, timed_ms: float, clocks) -> dict:
    """Which measured cuBLAS bf16 figure a tensor-bound number is compared with: the burst figure when the timed
    region is short (under about 2 s) or the SM clock stayed at its maximum, the sustained (power-capped) one
    otherwise."""
    sm, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    at_max = bool(sm and mx and sm >= 0.97 * mx)
    burst = timed_ms < 2000.0 or at_max
    return {"peak": peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"],
            "which": "burst" if burst else "sustained"}


def measure_step(m, args, world, rank, local, steps: int, graph: bool = True):
    """Times `steps` passes of the whole hot path of model `m` (device-resident inputs), CUDA events on the launching
    stream, barrier and synchronize on both sides of every timed region.
    Region 1 (the step): score + select + compact, then every layer's block (projections, attention core, FFN, and
      their backward) -> ms_step, ms_sp (the sparsify phase), ms_blocks.
    Region 2: the projection / FFN products of every layer on their own (the launches of gemm_kernel) -> ms_gemm.
    Region 3: the attention calls of every layer on their own -> ms_attn.
    Each region has its own clock record; `launches` counts the library's launches of one step of region 1."""
    import torch
    import torch.distributed as dist
    B = m.B
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    full = m.blocks if m.has_attention else m.layers
    for _ in range(max(3, args.warmup)):
        m.sparsify(); full(); m.layers()
    B.ecospa_device_status()
    # The calls are stateless and asynchronous, so a step can be captured once into CUDA graphs and
    # replayed: the launches of a step then cost no host time.  --no-graph issues them one by one.
    l0 = B.ecospa_launch_count()
    fns = {"sparsify": m.sparsify, "blocks": full, "gemm": m.layers}
    if m.has_attention:
        fns["attn"] = m.attention_only
    if not graph:
        m.sparsify(); full()
        launches = B.ecospa_launch_count() - l0
    else:
        graphs = {}
        for nm in ("sparsify", "blocks"):
            graphs[nm] = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graphs[nm]):
                fns[nm]()
        launches = B.ecospa_launch_count() - l0
        for nm in fns:
            if nm not in graphs:
                graphs[nm] = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graphs[nm]):
                    fns[nm]()
        fns = {nm: g.replay for nm, g in graphs.items()}
        m._graphs = graphs
    for _ in range(2):
        fns["sparsify"](); fns["blocks"]()
    B.ecospa_device_status()

    def region(seq_of_fns):
        """steps x the given calls; returns (ms per step of the whole, ms per step of each call, clock record)."""
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        marks = []
        barrier()
        t0, t1 = ev(), ev()
        t0.record()
        for _ in range(steps):
            es = [ev()]
            es[0].record()
            for f in seq_of_fns:
                f()
                es.append(ev()); es[-1].record()
            marks.append(es)
        t1.record()
        barrier()
        clocks = sampler.stop() if rank == 0 else None
        B.ecospa_device_status()
        parts = [sum(es[i].elapsed_time(es[i + 1]) for es in marks) / steps for i in range(len(seq_of_fns))]
        return t0.elapsed_time(t1) / steps, parts, clocks, t0.elapsed_time(t1)

    ms_step, (ms_sp, ms_blocks), clocks, timed_ms = region([fns["sparsify"], fns["blocks"]])
    ms_gemm, _, clocks_gemm, timed_gemm = region([fns["gemm"]])
    ms_attn, clocks_attn = None, None
    if "attn" in fns:
        ms_attn, _, clocks_attn, _ = region([fns["attn"]])
    return {"ms_step": ms_step, "ms_sp": ms_sp, "ms_blocks": ms_blocks, "ms_gemm": ms_gemm, "ms_attn": ms_attn,
            "clocks": clocks, "clocks_gemm": clocks_gemm, "clocks_attn": clocks_attn, "launches": int(launches),
            "replay": (fns["sparsify"], fns["blocks"]), "timed_ms": timed_ms, "timed_gemm_ms": timed_gemm}


def attention_report(wl, m, r):
    """The attention core's share: algorithmic flops / its own replay time, and its exponentials against the
    special-function rate of the part (one 2^x per query-key pair in the forward pass and in each of the two backward
    kernels; 16 per clock per SM, 148 SMs, at the SM clock sampled during the region)."""
    if r["ms_attn"] is None:
        return None
    fl = attention_flops(wl, m.plan["qk"][0], m.plan["vo"][0], m.causal)
    pairs = wl.batch * wl.n_heads * float(wl.seq) * wl.seq * (0.5 if m.causal else 1.0) * wl.n_layers
    sm = (r["clocks_attn"] or {}).get("sm_mhz") or 1965.0
    exp_peak = 148 * 16 * sm * 1e6          # exponentials per second
    return {"ms": r["ms_attn"], "TFLOP/s": fl / r["ms_attn"] / 1e9, "flops": fl, "frac_of_nominal_2250": fl / r["ms_attn"] / 1e9 / 2250.0,
            "causal": m.causal, "head_widths": f"{m.plan['qk'][0]} of {wl.d_h} (padded to {m.qk_w[0]})",
            "roofline": {"bound": "alu", "kernel": ("attn_fwd_ms_kernel" if max(m.vo_w) <= 32 and max(m.qk_w) <= 64 else "attn_fwd_kernel") + " + attn_bwd_kernel x2", "achieved": 3 * pairs / (r["ms_attn"] * 1e-3) / 1e12,
                         "peak": exp_peak / 1e12, "unit": "T exp/s", "frac": 3 * pairs / (r["ms_attn"] * 1e-3) / exp_peak,
                         "peak_source": f"16 ex2/clk/SM x 148 SMs x {sm:.0f} MHz (sampled)"},
            "clocks": r["clocks_attn"]}


def phase_report(wl, m, r, peaks, sparsity, transposed=False):
    """The figures of one measured workload: both phases against the measured and the nominal peaks."""
    flops = step_flops(wl, m.n_attn, m.k_ffn)
    sbytes = sparsify_bytes(wl, 1.0 - sparsity, transposed=transposed)
    tf = flops / r["ms_gemm"] / 1e9
    gbs = sbytes / r["ms_sp"] / 1e6
    tp = tensor_peak(peaks, r["timed_gemm_ms"], r["clocks_gemm"])
    sm = (r["clocks_gemm"] or {}).get("sm_mhz")
    afl = attention_flops(wl, m.plan["qk"][0], m.plan["vo"][0], m.causal) if m.has_attention else 0.0
    return {
        "workload": wl.name, "sparsity": sparsity, "ms_per_step": r["ms_step"],
        "step_TFLOP/s": (flops + afl) / r["ms_step"] / 1e9, "blocks_ms": r["ms_blocks"],
        "attention": attention_report(wl, m, r), "clocks_gemm": r["clocks_gemm"],
        "gemm_ms": r["ms_gemm"], "gemm_TFLOP/s": tf, "gemm_flops_per_step": flops,
        "gemm_frac_of_measured_burst": tf / peaks["bf16_tflops"],
        "gemm_frac_of_measured_sustained": tf / peaks["bf16_tflops_sustained"],
        "gemm_frac_of_nominal_2250": tf / 2250.0, "gemm_denominator_for_this_run": tp["which"],
        "gemm_ms_x_sm_mhz": (r["ms_gemm"] * sm) if sm else None,
        "sparsify_ms": r["ms_sp"], "sparsify_GB/s": gbs, "sparsify_bytes_per_step": sbytes,
        "sparsify_byte_accounting": "per tensor: every weight and gradient read once for the scores; compaction reads a "
                                    "shared-cols tensor in full and a shared-rows tensor at the kept fraction, writes the kept fraction",
        "sparsify_GB/s_if_every_tensor_counted_as_shared_rows": (2.0 + 4.0 * (1.0 - sparsity)) * WL_model_bytes(wl) / r["ms_sp"] / 1e6,
        "sparsify_frac_of_measured_hbm": gbs / peaks["hbm_gbs"], "sparsify_frac_of_nominal_8TBs": gbs / 8000.0,
        "clocks": r["clocks"], "gpu_launches": r["launches"],
    }


def WL_model_bytes(wl):
    from paper_2511_11641_b200 import workloads as WL
    return WL.model_bytes(wl)


# ---------------------------------------------------------------------------------------------
# the re-estimation sweep: score + select + compact over all layers at sparsity 10 ... 90 %, gradients redrawn
# per step with seeds 0 ... 9 (the per-epoch re-estimation of Algorithm 1); GB/s per sparsity, median over seeds
# ---------------------------------------------------------------------------------------------

def reestimation_sweep(wl, dev, local, rank, seeds=range(10), sparsities=tuple(s / 10 for s in range(1, 10)), reps=3):
    import torch
    from paper_2511_11641_b200 import binding as B, block as BL, workloads as WL
    w, g, pairs = [], [], []
    for l in range(wl.n_layers):
        w.append(WL.layer_weights(wl, l, device=dev))
        g.append(WL.layer_grads(wl, l, device=dev))
        pairs += BL.block_pairs(w[l], wl.n_heads, wl.d_h, wl.d_ffn, g[l])
    D_layer = 2 * wl.n_heads * wl.d_h + wl.d_ffn
    ups = torch.empty(D_layer * wl.n_layers, dtype=torch.float32, device=dev)
    fis = torch.empty((2 * wl.n_heads + 1) * wl.n_layers, dtype=torch.float32, device=dev)
    score_ws = torch.empty(B.ecospa_score_workspace_bytes(pairs), dtype=torch.uint8, device=dev)
    n_seg = [wl.n_heads, wl.n_heads, 1] * wl.n_layers
    seg_len = [wl.d_h, wl.d_h, wl.d_ffn] * wl.n_layers
    D_attn = wl.n_heads * wl.d_h
    layout = {"wq": 0, "wk": 0, "wv": 0, "wo": 1, "w1": 0, "w1b": 0, "w2": 1, "gq": 0, "gk": 0, "gv": 0, "go": 1, "g1": 0,
              "g1b": 0, "g2": 1}
    setups = {}
    for s in sparsities:
        plan = WL.kept_plan(wl, s)
        n_attn, k_ffn = sum(plan["qk"]), plan["ffn"][0]
        k_per_seg = (plan["qk"] + plan["vo"] + plan["ffn"]) * wl.n_layers
        kept = torch.empty(sum(k_per_seg), dtype=torch.int32, device=dev)
        jobs, outs, off = [], [], 0
        for l in range(wl.n_layers):
            for names, nk, D in ((("wq", "wk", "gq", "gk"), n_attn, D_attn), (("wv", "wo", "gv", "go"), n_attn, D_attn),
                                 (("w1", "w1b", "w2", "g1", "g1b", "g2"), k_ffn, wl.d_ffn)):
                kd = kept[off:off + nk]
                for nm in names:
                    src = w[l].get(nm) if nm in w[l] else g[l].get(nm)
                    if src is None:
                        continue
                    o = BL.alloc_compacted(src, layout[nm], nk)
                    outs.append(o)
                    jobs.append(B.gather(src, o, layout[nm], kd, nk, D))
                off += nk
        setups[s] = (k_per_seg, kept, jobs, outs)

    def run(s):
        k_per_seg, kept, jobs, _ = setups[s]
        B.ecospa_score_pairs(pairs, float(wl.tokens), ups, None, fis, score_ws)
        B.ecospa_select_aligned_topk(ups, n_seg, seg_len, k_per_seg, kept)
        B.ecospa_compact_tensors(jobs)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    times = {s: [] for s in sparsities}
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for s in sparsities:
        run(s)                                                       # warm-up of every configuration
    torch.cuda.synchronize()
    fisher_by_seed = []
    for seed in seeds:
        for l in range(wl.n_layers):                                 # redraw the gradients of this step, in place
            fresh = WL.layer_grads(wl, l, step=seed, device=dev)
            for nm, t in fresh.items():
                g[l][nm].copy_(t)
            del fresh
        for s in sparsities:
            run(s)
            e0, e1 = ev(), ev()
            e0.record()
            for _ in range(reps):
                run(s)
            e1.record()
            torch.cuda.synchronize()
            times[s].append(e0.elapsed_time(e1) / reps)
        fisher_by_seed.append(float(fis.double().mean().item()))
    clocks = sampler.stop() if rank == 0 else None
    B.ecospa_device_status()
    peaks = measured_peaks()
    out = {"workload": wl.name, "seeds": len(list(seeds)), "reps_per_seed": reps, "clocks": clocks, "per_sparsity": {}}
    for s in sparsities:
        ms = statistics.median(times[s])
        by = sparsify_bytes(wl, 1.0 - s)
        out["per_sparsity"][f"{s:.1f}"] = {"ms_median": ms, "GB/s": by / ms / 1e6, "bytes": by,
                                          "frac_of_measured_hbm": by / ms / 1e6 / peaks["hbm_gbs"],
                                          "frac_of_nominal_8TBs": by / ms / 1e6 / 8000.0}
    # the importance values do change from draw to draw (the scores do not depend on the gradients)
    out["mean_importance_by_seed_distinct"] = len(set(fisher_by_seed)) == len(fisher_by_seed)
    return out


# ---------------------------------------------------------------------------------------------
# parity of what was timed: layer 0 of the benchmarked model against the oracle
# ---------------------------------------------------------------------------------------------

def parity_check(m, n_rows: int = 8):
    """Re-runs the step's calls on layer 0 of the benchmarked model and compares them with the CPU oracle: scores,
    kept sets (oracle ranking of the same fp32 scores), compacted weights (bytes), and the layer outputs and input
    gradients on sampled token rows (relative l2 per row, fp64 oracle)."""
    import numpy as np
    import torch
    from oracle import oracle as O
    wl, B = m.wl, m.B
    if m.transposed:
        return {"skipped": "weights stored transposed: the tests cover this orientation"}
    m.sparsify()
    m.o["dX"].zero_()
    m.layer(0)
    B.ecospa_device_status()
    kept_p_all = m.kept_p.cpu().numpy() if m.padded else None
    w = {k: v.cpu() for k, v in m.w[0].items()}
    D_attn = wl.n_heads * wl.d_h
    D_layer = 2 * D_attn + wl.d_ffn
    ups = m.ups[:D_layer].cpu().numpy()
    sw = wl.ffn == "swiglu"
    groups = [("wq", "wk", None, 0, 0, wl.n_heads, wl.d_h, m.plan["qk"]), ("wv", "wo", None, 0, 1, wl.n_heads, wl.d_h, m.plan["vo"]),
              ("w1", "w2", "w1b" if sw else None, 0, 1, 1, wl.d_ffn, m.plan["ffn"])]
    res = {"tolerance_rows": 2e-2, "tolerance_scores": 1e-5}
    off_d, off_k, score_err, kept_equal, bytes_equal = 0, 0, 0.0, True, True
    kept_all = m.kept.cpu().numpy()
    kept_of = {}
    for n1, n2, n1b, l1, l2, n_seg, seg_len, k in groups:
        _, ups_o = O.score_pair(w[n1], w[n2], l1, l2, n_seg, seg_len, w1b=w.get(n1b) if n1b else None)
        got = ups[off_d:off_d + n_seg * seg_len].astype(np.float64)
        for sgm in range(n_seg):
            a, b = sgm * seg_len, (sgm + 1) * seg_len
            score_err = max(score_err, float(np.max(np.abs(got[a:b] - ups_o[a:b]) / (np.abs(ups_o[a:b]) + ups_o[a:b].max()))))
        kept_o = O.select_topk(ups[off_d:off_d + n_seg * seg_len], n_seg, seg_len, k)
        kept_g = kept_all[off_k:off_k + sum(k)]
        kept_equal = kept_equal and bool(np.array_equal(kept_o, kept_g))
        if m.padded and n_seg > 1:
            # the list the compaction used: every head's kept indices followed by "no index" entries up to its padded width
            gi = 0 if n1 == "wq" else 1
            kept_g = kept_p_all[gi * m.n_attn_p:(gi + 1) * m.n_attn_p]
            widths = m.qk_w if gi == 0 else m.vo_w
            exp = np.concatenate([np.concatenate([kept_o[sum(k[:h]):sum(k[:h + 1])], -np.ones(widths[h] - k[h], dtype=np.int32)])
                                  for h in range(n_seg)])
            kept_equal = kept_equal and bool(np.array_equal(exp, kept_g))
        kept_of[n1] = kept_g
        for nm, lay in ((n1, l1), (n2, l2), (n1b, l1)):
            if nm:
                o = m.c[0][nm]
                ref = O.compact(w[nm], lay, kept_g, ld_out=o.shape[1])
                bytes_equal = bytes_equal and bool(torch.equal(o.cpu().view(torch.int16), ref.view(torch.int16)))
        off_d += n_seg * seg_len; off_k += sum(k)
    res.update({"score_max_rel_err": score_err, "kept_sets_equal": kept_equal, "compacted_bytes_equal": bytes_equal})
    # layer math on sampled token rows
    r = np.random.default_rng(0)
    rows = np.sort(r.choice(wl.tokens, size=n_rows, replace=False))
    rt = torch.from_numpy(rows); rd = rt.to(m.dev)
    a = m.acts[0]
    c = {k: v.cpu() for k, v in m.c[0].items() if k in ("wq", "wk", "wv", "wo", "w1", "w1b", "w2", "bq", "bk", "bv", "b1")}
    n, k = m.n_attn_p, m.k_ffn
    X = a["x"][rd].cpu().contiguous()

    def row_err(got, ref):
        got = got.double().cpu().numpy()
        return float(np.max(np.linalg.norm(got - ref, axis=1) / np.maximum(np.linalg.norm(ref, axis=1), 1e-300)))

    errs = {}
    for nm, out in (("q", "Q"), ("k", "K"), ("v", "V")):
        errs[out] = row_err(m.o[out][rd][:, :n], O.proj_fwd(X, c["w" + nm], 0, n, bias=c.get("b" + nm)))
    ctx = a["ctx"][rd].cpu()[:, :n].contiguous()
    errs["Out"] = row_err(m.o["Out"][rd], O.outproj_fwd(ctx, c["wo"], 1, n, wl.d_m))
    rdCtx, _, _ = O.outproj_bwd(ctx, c["wo"], 1, n, wl.d_m, a["dout"][rd].cpu().contiguous())
    errs["dCtx"] = row_err(m.o["dCtx"][rd][:, :n], rdCtx)
    rdX = None
    for nm in ("q", "k", "v"):
        rdX, _, _ = O.proj_bwd(X, c["w" + nm], 0, n, a["d" + nm][rd].cpu()[:, :n].contiguous(), dX=rdX)
    errs["dX(attention)"] = row_err(m.o["dX"][rd], rdX)
    act = O.ACT_SWIGLU if sw else O.ACT_GELU_ERF
    b2 = w.get("b2")
    rf = O.ffn_fwd(X, act, c["w1"], c["w2"], 0, 1, k, W1b=c.get("w1b"), b1=c.get("b1"), b2=b2)
    rb = O.ffn_bwd(X, act, c["w1"], c["w2"], 0, 1, k, a["dy"][rd].cpu().contiguous(), W1b=c.get("w1b"), b1=c.get("b1"))
    errs["Y"] = row_err(m.ffn["Y"][rd], rf["Y"])
    errs["A"] = row_err(m.ffn["A"][rd][:, :k], rf["A"])
    errs["dX(ffn)"] = row_err(m.ffn["dX"][rd], rb["dX"])
    res["max_row_rel_err"] = errs
    res["rows_sampled"] = int(n_rows)
    aerrs = {}
    if m.has_attention:
        # the chained block of layer 0, then one (sequence, head) pair of its attention core against the oracle
        m.block(0)
        B.ecospa_device_status()
        b_s, h_s = wl.batch - 1, min(3, wl.n_heads - 1)
        rows_s = slice(b_s * wl.seq, (b_s + 1) * wl.seq)
        kq, kv = m.plan["qk"][h_s], m.plan["vo"][h_s]
        cq = slice(m.qk_off[h_s], m.qk_off[h_s] + kq)
        cv = slice(m.vo_off[h_s], m.vo_off[h_s] + kv)
        sub = lambda t, c: t[rows_s, c].cpu().contiguous()
        q, kk_, v, dc = sub(m.o["Q"], cq), sub(m.o["K"], cq), sub(m.o["V"], cv), sub(m.o["dCtx"], cv)
        rf = O.attn_fwd(q, kk_, v, 1, wl.seq, [0], [kq], [0], [kv], m.scale, m.causal)
        rb = O.attn_bwd(q, kk_, v, dc, 1, wl.seq, [0], [kq], [0], [kv], m.scale, m.causal)
        fro = lambda got, ref: float(np.linalg.norm(got.double().cpu().numpy() - ref) / max(np.linalg.norm(ref), 1e-300))
        aerrs = {"Ctx": fro(m.o["Ctx"][rows_s, cv], rf["Ctx"]), "dQ": fro(m.o["dQ"][rows_s, cq], rb["dQ"]),
                 "dK": fro(m.o["dK"][rows_s, cq], rb["dK"]), "dV": fro(m.o["dV"][rows_s, cv], rb["dV"])}
        res["attention_rel_frobenius"] = aerrs
        res["attention_sample"] = f"sequence {b_s}, head {h_s} of layer 0, in full"
    res["ok"] = bool(kept_equal and bytes_equal and score_err <= 1e-5 and all(v <= 2e-2 for v in errs.values())
                     and all(v <= 2e-2 for v in aerrs.values()))
    return res


def run_gpu(args):
    import dataclasses
    import torch
    import torch.distributed as dist
    from paper_2511_11641_b200 import binding as B, workloads as WL
    import __graft_entry__ as ge
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0:
        ge.build()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    dev = torch.device("cuda", local)
    wl = WL.WORKLOADS[args.workload]
    if args.layers:
        wl = dataclasses.replace(wl, n_layers=args.layers)   # smaller model of the same shape (profiler captures)
    m = Model(wl, args.sparsity, dev, transposed=args.transposed)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    r = measure_step(m, args, world, rank, local, args.steps, graph=not args.no_graph)
    sparsify, layers = r["replay"]
    ms_step, ms_sp, ms_gemm, clocks, launches = r["ms_step"], r["ms_sp"], r["ms_gemm"], r["clocks"], r["launches"]

    # ---- end to end: every step's inputs start in pinned host memory and its results are read back.
    # Two device-side copies of the model take turns, so the upload of step s + 1 (copy stream) runs while
    # step s computes; every step still pays its own upload and read-back inside the timed region.
    host = m.host_copies()
    h2d = sum(h.numel() * h.element_size() for h, _ in host)
    m2 = Model(wl, args.sparsity, dev, transposed=args.transposed)
    full2 = m2.blocks if m2.has_attention else m2.layers
    for _ in range(3):
        m2.sparsify(); full2()
    if args.no_graph:
        replay = [(sparsify, layers), (m2.sparsify, full2)]
    else:
        g2_sp, g2_ly = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2_sp):
            m2.sparsify()
        with torch.cuda.graph(g2_ly):
            full2()
        replay = [(sparsify, layers), (g2_sp.replay, g2_ly.replay)]
    models = [m, m2]
    dev_in = [[d for _, d in host], [t for dd in m2.w + m2.g + m2.acts for t in dd.values()]]
    host_in = [h for h, _ in host]
    assert all(a.shape == b.shape and a.dtype == b.dtype for a, b in zip(dev_in[0], dev_in[1]))
    res_host = [[torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in (mm.kept, mm.fis, mm.ups)] for mm in models]
    chk_host = torch.empty(2, dtype=torch.float32, pin_memory=True)
    d2h = sum(t.numel() * t.element_size() for t in res_host[0]) + 4
    copy_stream = torch.cuda.Stream(device=dev)
    copied = [torch.cuda.Event(), torch.cuda.Event()]
    done = [torch.cuda.Event(), torch.cuda.Event()]

    def e2e_steps_run(n):
        cur = torch.cuda.current_stream()
        for s_i in range(n):
            b = s_i % 2
            mm = models[b]
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(done[b])               # the previous step on this copy of the model is over
                for h, d in zip(host_in, dev_in[b]):
                    d.copy_(h, non_blocking=True)
                copied[b].record(copy_stream)
            cur.wait_event(copied[b])
            replay[b][0](); replay[b][1]()
            for h, d in zip(res_host[b], (mm.kept, mm.fis, mm.ups)):
                h.copy_(d, non_blocking=True)
            chk_host[b:b + 1].copy_(mm.o["dX"][0, :1].float(), non_blocking=True)
            done[b].record(cur)

    e2e_steps = max(4, min(args.steps, 8))
    e2e_steps_run(2)
    barrier()
    e0, e1 = ev(), ev()
    e0.record()
    e2e_steps_run(e2e_steps)
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1) / e2e_steps
    B.ecospa_device_status()
    del m2, host, host_in, dev_in, res_host, replay
    if not args.no_graph:
        del g2_sp, g2_ly

    ms_attn = r["ms_attn"] if r["ms_attn"] is not None else 0.0
    ms_step, ms_sp, ms_gemm, ms_e2e, ms_attn, ms_blocks = max_over_ranks([ms_step, ms_sp, ms_gemm, ms_e2e, ms_attn, r["ms_blocks"]], dev)
    r["ms_gemm"], r["ms_sp"], r["ms_step"], r["ms_blocks"] = ms_gemm, ms_sp, ms_step, ms_blocks
    if r["ms_attn"] is not None:
        r["ms_attn"] = ms_attn

    gemm_flops = step_flops(wl, m.n_attn, m.k_ffn)
    attn_flops = attention_flops(wl, m.plan["qk"][0], m.plan["vo"][0], m.causal) if m.has_attention else 0.0
    flops = gemm_flops + attn_flops            # every product of a step: projections, FFN, attention core
    sbytes = sparsify_bytes(wl, 1.0 - args.sparsity, transposed=args.transposed)
    peaks = measured_peaks()
    n_gemm_launches = wl.n_layers * 8
    tf = gemm_flops / ms_gemm / 1e9
    tp = tensor_peak(peaks, r["timed_gemm_ms"], r["clocks_gemm"])
    sm_mhz = (r["clocks_gemm"] or {}).get("sm_mhz")
    plain = not args.layers and args.sparsity == 0.5 and not args.transposed
    sp_traffic = NCU_SPARSIFY_TRAFFIC_BYTES_PER_LAYER.get(wl.name)
    out = {
        "metric": METRIC, "value": job_throughput(world, flops, ms_step) / 1e9, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic (seeded N(0,sigma) tensors)",
        "config": {"workload": f"{wl.name}: {wl.n_layers} layers d_model={wl.d_m} heads={wl.n_heads}x{wl.d_h} "
                               f"ffn={wl.d_ffn} {wl.ffn} T={wl.tokens} sparsity={args.sparsity}"
                               + (" weights stored transposed" if args.transposed else ""),
                   "l2": f"inputs larger than L2: {2 * WL.model_bytes(wl) / 1e9:.1f} GB of weights/gradients per step, "
                         "activations cycled over 4 sets",
                   "replicas": world, "launch": "eager" if args.no_graph else "cuda graph replay of the captured step"},
        "phases": {
            "sparsify": {"ms": ms_sp, "GB/s": sbytes / ms_sp / 1e6, "bytes": sbytes,
                         "byte_accounting": "per tensor (scores: every weight and gradient once; compaction: shared-cols "
                                            "tensors read in full, shared-rows at the kept fraction, kept fraction written)",
                         "GB/s_if_every_tensor_counted_as_shared_rows": (2.0 + 4.0 * (1.0 - args.sparsity)) * WL.model_bytes(wl) / ms_sp / 1e6,
                         "frac_of_measured_hbm": sbytes / ms_sp / 1e6 / peaks["hbm_gbs"],
                         "frac_of_nominal_8TBs": sbytes / ms_sp / 1e6 / 8000.0},
            "blocks": {"ms": ms_blocks, "what": "every layer's projections, attention core, FFN and their backward, chained",
                       "TFLOP/s": flops / ms_blocks / 1e9},
            "attention": attention_report(wl, m, r),
            "gemm": {"ms": ms_gemm, "TFLOP/s": tf, "flops": gemm_flops, "clocks": r["clocks_gemm"],
                     "what": "the projection and FFN products of every layer replayed on their own (gemm_kernel launches)",
                     "frac_of_measured_burst": tf / peaks["bf16_tflops"],
                     "frac_of_measured_sustained": tf / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": tf / 2250.0,
                     "ms_x_sm_mhz": ms_gemm * sm_mhz if sm_mhz else None},
        },
        # the layer phase = 8 gemm_kernel launches per layer plus the small bias-gradient / split-K finishing launches,
        # so `achieved` slightly understates the kernel itself
        "roofline": {"bound": "tensor", "kernel": "gemm_kernel", "achieved": tf,
                     "peak": tp["peak"], "unit": "TFLOP/s", "frac": tf / tp["peak"],
                     "peak_source": f"{peaks['source']} cuBLAS bf16, {tp['which']} figure (timed region "
                                    f"{r['timed_gemm_ms'] / 1e3:.2f} s, median SM clock {sm_mhz} MHz)",
                     "frac_of_measured_burst": tf / peaks["bf16_tflops"],
                     "frac_of_measured_sustained": tf / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": tf / 2250.0,
                     "traffic": NCU_GEMM_TRAFFIC_BYTES.get(wl.name) if plain else None,
                     "traffic_unit": "bytes per launch (DRAM read + write, ncu)",
                     "launches_per_step": n_gemm_launches, "avg_launch_ms": ms_gemm / n_gemm_launches},
        # the memory-bound part of the step against the measured copy bandwidth: score + select + compact as one unit
        # (sumsq_kernel and gather_kernel move all of its bytes; traffic = their DRAM bytes under ncu, which grow in
        # proportion to the layer count)
        "roofline_hbm": {"bound": "hbm", "kernel": "sumsq_kernel + gather_kernel (+ finalize, select)",
                         "achieved": sbytes / ms_sp / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": sbytes / ms_sp / 1e6 / peaks["hbm_gbs"],
                         "frac_of_nominal_8TBs": sbytes / ms_sp / 1e6 / 8000.0,
                         "traffic": sp_traffic * wl.n_layers if (sp_traffic and plain) else None,
                         "traffic_unit": "bytes per step (DRAM read + write, ncu, scaled by layers)",
                         "peak_source": peaks["source"] + " (copy bandwidth)"},
        "e2e": {"value": job_throughput(world, flops, ms_e2e) / 1e9, "unit": "TFLOP/s", "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipeline": "two device copies of the model: the upload of step s+1 overlaps the compute of step s"},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    if rank == 0 and world == 1:
        out["parity_check"] = parity_check(m)
    # ---- the other configurations (1 GPU runs only): each with its own clock record
    if world == 1 and not args.no_configs and not args.layers:
        cfgs = {}
        cfgs["cfg3_llama1b" if wl.name == "llama1b" else "main"] = phase_report(wl, m, r, peaks, args.sparsity, args.transposed)
        del m, sparsify, layers, r
        torch.cuda.empty_cache()
        cfg_steps = {"gpt2m": 40, "llama1b": 20, "llama7b_layer": 60}
        plan = [("cfg2_gpt2m", "gpt2m", 0.5), ("cfg3_llama1b", "llama1b", 0.5), ("cfg4_llama7b_layer_s0.25", "llama7b_layer", 0.25),
                ("cfg4_llama7b_layer_s0.50", "llama7b_layer", 0.5), ("cfg4_llama7b_layer_s0.75", "llama7b_layer", 0.75)]
        for key, name, sp in plan:
            if key in cfgs:
                continue
            w2 = WL.WORKLOADS[name]
            mm = Model(w2, sp, dev)
            rr = measure_step(mm, args, world, rank, local, cfg_steps[name], graph=not args.no_graph)
            cfgs[key] = phase_report(w2, mm, rr, peaks, sp)
            del mm, rr
            torch.cuda.empty_cache()
        cfgs["cfg5_reestimation_sweep"] = reestimation_sweep(WL.WORKLOADS["llama1b"], dev, local, rank)
        torch.cuda.empty_cache()
        out["configs"] = cfgs
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(wl, args.sparsity)
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# the CPU oracle on a bounded sample of the same step
# ---------------------------------------------------------------------------------------------

def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def cpu_sample(wl, sparsity: float, tokens: int = 256, threads: int = 1):
    """Layer 0 of the workload through the oracle, as it stands: score + Fisher + select + compact at full size,
    then forward/backward of the compacted pairs on `tokens` token rows.  With threads > 1 the pair groups (and their
    tensors) of the first part, and equal chunks of the token rows of the second, are handed to a thread pool (the
    oracle's C routines release the interpreter lock); every thread runs the same plain code on its share.  Returns
    the metric (algorithmic flops / wall time) for that sample."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle as O
    from paper_2511_11641_b200 import workloads as WL
    from paper_2511_11641_b200.block import pad8
    w = WL.layer_weights(wl, 0)
    g = WL.layer_grads(wl, 0)
    plan = WL.kept_plan(wl, sparsity)
    n_attn, k_ffn = sum(plan["qk"]), plan["ffn"][0]
    acts = WL.activations(wl, 0, tokens=tokens, kinds=["x", "dy", "dout", "dq", "dk", "dv", "ctx"],
                          widths={kk: n_attn for kk in ("dq", "dk", "dv", "ctx")})
    sw = wl.ffn == "swiglu"
    act = O.ACT_SWIGLU if sw else O.ACT_GELU_ERF
    pool = ThreadPoolExecutor(max_workers=threads) if threads > 1 else None

    def run_all(fns):
        if pool is None:
            return [f() for f in fns]
        return [fu.result() for fu in [pool.submit(f) for f in fns]]

    t0 = time.perf_counter()
    groups = [("wq", "wk", None, "gq", "gk", None, 0, 0, wl.n_heads, wl.d_h, plan["qk"]),
              ("wv", "wo", None, "gv", "go", None, 0, 1, wl.n_heads, wl.d_h, plan["vo"]),
              ("w1", "w2", "w1b" if sw else None, "g1", "g2", "g1b" if sw else None, 0, 1, 1, wl.d_ffn, plan["ffn"])]
    c = {}

    def do_group(grp):
        n1, n2, n1b, g1, g2, g1b, l1, l2, n_seg, seg_len, k = grp
        _, ups = O.score_pair(w[n1], w[n2], l1, l2, n_seg, seg_len, w1b=w.get(n1b) if n1b else None)
        O.fisher_pair(g[g1], g[g2], l1, l2, n_seg, seg_len, float(wl.tokens), g1b=g.get(g1b) if g1b else None)
        kept = O.select_topk(ups.astype(np.float32), n_seg, seg_len, k)
        out = {}
        for nm, lay in ((n1, l1), (n2, l2), (n1b, l1), (g1, l1), (g2, l2), (g1b, l1)):
            if nm:
                src = w[nm] if nm in w else g[nm]
                out[nm] = O.compact(src, lay, kept, ld_out=pad8(len(kept), wl.elem_bytes) if lay == 0 else None)
        return out

    for d in run_all([(lambda grp=grp: do_group(grp)) for grp in groups]):
        c.update(d)
    t1 = time.perf_counter()

    def do_rows(lo, hi):
        x = acts["x"][lo:hi].contiguous()
        sl = lambda nm: acts[nm][lo:hi].contiguous()
        O.proj_fwd(x, c["wq"], 0, n_attn); O.proj_fwd(x, c["wk"], 0, n_attn); O.proj_fwd(x, c["wv"], 0, n_attn)
        O.outproj_fwd(sl("ctx"), c["wo"], 1, n_attn, wl.d_m)
        dX, _, _ = O.proj_bwd(x, c["wq"], 0, n_attn, sl("dq"))
        O.proj_bwd(x, c["wk"], 0, n_attn, sl("dk"), dX=dX)
        O.proj_bwd(x, c["wv"], 0, n_attn, sl("dv"))
        O.outproj_bwd(sl("ctx"), c["wo"], 1, n_attn, wl.d_m, sl("dout"))
        O.ffn_fwd(x, act, c["w1"], c["w2"], 0, 1, k_ffn, W1b=c.get("w1b"))
        O.ffn_bwd(x, act, c["w1"], c["w2"], 0, 1, k_ffn, sl("dy"), W1b=c.get("w1b"))

    chunks = max(1, min(threads, tokens))
    bounds = [(i * tokens // chunks, (i + 1) * tokens // chunks) for i in range(chunks)]
    run_all([(lambda lo=lo, hi=hi: do_rows(lo, hi)) for lo, hi in bounds if hi > lo])
    # attention core: `threads` heads of one sequence truncated to s_a positions (causal), forward and backward
    s_a = min(wl.seq, 256)
    kq, kv = plan["qk"][0], plan["vo"][0]
    aw = WL.activations(wl, 1, tokens=s_a, kinds=["dq", "dk", "dv", "ctx"], widths={kk: kq for kk in ("dq", "dk")} | {"dv": kv, "ctx": kv})

    def do_head():
        O.attn_fwd(aw["dq"], aw["dk"], aw["dv"], 1, s_a, [0], [kq], [0], [kv], 1.0 / wl.d_h ** 0.5, True)
        O.attn_bwd(aw["dq"], aw["dk"], aw["dv"], aw["ctx"], 1, s_a, [0], [kq], [0], [kv], 1.0 / wl.d_h ** 0.5, True)

    n_heads_a = max(1, threads)
    run_all([do_head for _ in range(n_heads_a)])
    t2 = time.perf_counter()
    if pool is not None:
        pool.shutdown()
    attn_fl = n_heads_a * 0.5 * s_a * s_a * 2.0 * ((kq + kv) + (3 * kq + 2 * kv))
    flops = step_flops(wl, n_attn, k_ffn) / wl.n_layers * tokens / wl.tokens + attn_fl
    sbytes = sparsify_bytes(wl, 1.0 - sparsity) / wl.n_layers
    return {"value": flops / (t2 - t0) / 1e12, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
            "sample": f"layer 0 of {wl.name}: score+Fisher+select+compact at full size ({t1 - t0:.2f} s, "
                      f"{sbytes / (t1 - t0) / 1e9:.3f} GB/s), then fwd+bwd of the compacted QK/VO/FFN pairs on "
                      f"{tokens} of {wl.tokens} tokens and of the attention core on {n_heads_a} head(s) x {s_a} positions "
                      f"({t2 - t1:.2f} s), {threads} thread(s)",
            "seconds": t2 - t0, "gemm_tflops": flops / (t2 - t1) / 1e12, "sparsify_GB/s": sbytes / (t1 - t0) / 1e9}


def sample_tokens(wl, seconds: float = 12.0) -> int:
    """Token rows whose fp64 triple-loop forward/backward takes about `seconds` on one core (~1.5 GFLOP/s)."""
    per_token = step_flops(wl, wl.n_heads * wl.d_h // 2, wl.d_ffn // 2) / wl.n_layers / wl.tokens
    return int(max(16, min(256, seconds * 1.5e9 / per_token)))


def cpu_baseline(wl, sparsity: float):
    """The oracle timed on this machine's host cores: once on one thread, once on every core of the affinity mask
    (capped at 32) on a sample of `cores` times as many token rows.  `value` / `cores` are the threaded run."""
    tokens = sample_tokens(wl)
    one = cpu_sample(wl, sparsity, tokens, threads=1)
    cores = min(32, host_cores())
    if cores == 1:
        one["single_thread"] = {"value": one["value"], "sample": one["sample"]}
        return one
    many = cpu_sample(wl, sparsity, min(wl.tokens, tokens * min(cores, 8)), threads=cores)
    many["single_thread"] = {"value": one["value"], "gemm_tflops": one["gemm_tflops"], "sparsify_GB/s": one["sparsify_GB/s"],
                             "sample": one["sample"]}
    many["host_cores_in_affinity_mask"] = host_cores()
    return many


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as O
    from paper_2511_11641_b200 import workloads as WL
    O.build()
    wl = WL.WORKLOADS[args.workload]
    tokens = 32
    steps, warm = max(1, min(args.steps, 5)), max(1, min(args.warmup, 1))
    for _ in range(warm):
        cpu_sample(wl, args.sparsity, tokens)
    t0 = time.perf_counter()
    last = None
    for _ in range(steps):
        last = cpu_sample(wl, args.sparsity, tokens)
    dt = (time.perf_counter() - t0) / steps
    v = last["value"] * last["seconds"] / dt     # the sample's flops over the mean step time
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic (seeded N(0,sigma) tensors)",
        "config": {"workload": f"{wl.name}: bounded sample of the step (layer 0, {tokens} of {wl.tokens} tokens), "
                               f"sparsity={args.sparsity}"},
        "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": 1, "kind": "oracle", "sample": last["sample"]},
        "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama1b")
    ap.add_argument("--sparsity", type=float, default=0.5)
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (small cases for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the other configurations (GPT-2-Medium shape, LLaMA-7B layer at three sparsities, "
                         "re-estimation sweep) that a 1-GPU run reports beside the main workload")
    ap.add_argument("--transposed", action="store_true",
                    help="store every weight matrix the other way round (W_Q.. as D x d_m, W_O, W_2 as d_m x D)")
    ap.add_argument("--no-graph", action="store_true", help="issue every launch from the host instead of replaying a CUDA graph")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
