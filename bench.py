"""Benchmark of the coupled-sparsity hot path on a GPT-2-Medium-shaped model (or another workload).

One step = one pass of the whole hot path over every layer of the model:
  score (+ Fisher) of all coupled pairs -> aligned top-k -> compaction of weights, biases and
  gradients -> forward and backward of every compacted QK / VO / FFN pair.

    python bench.py --gpus 1 --steps 10 --warmup 3
    python bench.py --impl reference            # the CPU oracle on a bounded sample of the same step

Prints one JSON line (rank 0).  `value` is the tensor-core throughput of the step (algorithmic
flops of the compacted-pair GEMMs / whole step time); the memory-bound phase is reported
alongside as GB/s.  With N > 1 every rank runs an independent replica (the path has no exchange
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

# DRAM bytes (read + write) per gemm_kernel launch, averaged over the eight GEMM launches of a gpt2m layer:
# `dram__bytes_read.sum + dram__bytes_write.sum` of one ncu capture of this build (profiles/gemm_kernel_gpt2m_layer.md).
# Per-launch traffic does not depend on the number of layers captured.  Other workloads: not captured (None).
NCU_GEMM_TRAFFIC_BYTES = {"gpt2m": 45.3e6}

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
        self.n_attn, self.k_ffn = sum(plan["qk"]), plan["ffn"][0]
        self.k_per_seg = (plan["qk"] + plan["vo"] + plan["ffn"]) * wl.n_layers
        self.n_seg = [wl.n_heads, wl.n_heads, 1] * wl.n_layers
        self.seg_len = [wl.d_h, wl.d_h, wl.d_ffn] * wl.n_layers
        D_layer = 2 * wl.n_heads * wl.d_h + wl.d_ffn
        f32, i32 = torch.float32, torch.int32
        self.ups = torch.empty(D_layer * wl.n_layers, dtype=f32, device=device)
        self.fis = torch.empty((2 * wl.n_heads + 1) * wl.n_layers, dtype=f32, device=device)
        self.kept = torch.empty(sum(self.k_per_seg), dtype=i32, device=device)
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
        for l in range(wl.n_layers):
            c = {}
            for wn, gn, nk, D in groups:
                kd = self.kept[off:off + nk]
                for nm in wn + gn:
                    src = self.w[l].get(nm) if nm in self.w[l] else self.g[l].get(nm)
                    if src is None:
                        continue
                    o = BL.alloc_compacted(src, layout[nm], nk)
                    c[nm] = o
                    self.jobs.append(B.gather(src, o, layout[nm], kd, nk, D))
                off += nk
            self.c.append(c)
        # activations and upstream gradients: a small pool of distinct sets cycled over the layers
        T, d, n, k = wl.tokens, wl.d_m, self.n_attn, self.k_ffn
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
        B.ecospa_compact_tensors(self.jobs)

    def layers(self):
        B, o, n, k = self.B, self.o, self.n_attn, self.k_ffn
        bias = self.wl.bias
        for l in range(self.wl.n_layers):
            c, a = self.c[l], self.acts[l % len(self.acts)]
            # forward: Q, K, V in one launch; (attention core is the caller's); output projection; FFN
            B.ecospa_coupled_qkv_fwd(a["x"], c["wq"], c["wk"], c["wv"], n, n, o["Q"], o["K"], o["V"], bq_c=c.get("bq"),
                                     bk_c=c.get("bk"), bv_c=c.get("bv"), workspace=self.proj_ws, **self.lay)
            B.ecospa_coupled_vo_fwd_o(a["ctx"], c["wo"], n, o["Out"], workspace=self.proj_ws, **self.lay)
            # FFN forward + backward
            self.L.ffn_fwd_bwd(a["x"], a["dy"], self.act, c["w1"], c["w2"], k, self.ffn, w1bc=c.get("w1b"),
                               b1c=c.get("b1"), b2=self.w[l].get("b2"), **self.lay)
            # backward: what dOut gives (dCtx, dW_O), then what dQ, dK, dV give (dW_Q, dW_K, dW_V, dX)
            B.ecospa_coupled_vo_bwd_o(a["ctx"], c["wo"], n, a["dout"], o["dCtx"], o["dWo"], o["dbo"] if bias else None,
                                      workspace=self.proj_ws, **self.lay)
            B.ecospa_coupled_qkv_bwd(a["x"], c["wq"], c["wk"], c["wv"], n, n, a["dq"], a["dk"], a["dv"], o["dX"], o["dWq"],
                                     o["dWk"], o["dWv"], o["dbq"] if bias else None, o["dbk"] if bias else None,
                                     o["dbv"] if bias else None, accumulate_dX=True, workspace=self.proj_ws, **self.lay)

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


def run_gpu(args):
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
        import dataclasses
        wl = dataclasses.replace(wl, n_layers=args.layers)   # smaller model of the same shape (profiler captures)
    m = Model(wl, args.sparsity, dev, transposed=args.transposed)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        m.sparsify(); m.layers()
    B.ecospa_device_status()
    # The calls are stateless and asynchronous, so a step can be captured once into CUDA graphs and
    # replayed: the ~500 launches of a step then cost no host time.  --no-graph issues them one by one.
    l0 = B.ecospa_launch_count()
    if args.no_graph:
        sparsify, layers = m.sparsify, m.layers
        m.sparsify(); m.layers()
    else:
        g_sp, g_ly = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_sp):
            m.sparsify()
        with torch.cuda.graph(g_ly):
            m.layers()
        sparsify, layers = g_sp.replay, g_ly.replay
    launches = B.ecospa_launch_count() - l0
    for _ in range(2):
        sparsify(); layers()
    B.ecospa_device_status()
    # ---- device-resident timing
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    marks = []
    barrier()
    t_all0, t_all1 = ev(), ev()
    t_all0.record()
    for _ in range(args.steps):
        e0, e1, e2 = ev(), ev(), ev()
        e0.record(); sparsify(); e1.record(); layers(); e2.record()
        marks.append((e0, e1, e2))
    t_all1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    B.ecospa_device_status()
    ms_total = t_all0.elapsed_time(t_all1)
    ms_sp = sum(a.elapsed_time(b) for a, b, _ in marks) / args.steps
    ms_gemm = sum(b.elapsed_time(c) for _, b, c in marks) / args.steps
    ms_step = ms_total / args.steps

    # ---- end to end: every step's inputs start in pinned host memory and its results are read back.
    # Two device-side copies of the model take turns, so the upload of step s + 1 (copy stream) runs while
    # step s computes; every step still pays its own upload and read-back inside the timed region.
    host = m.host_copies()
    h2d = sum(h.numel() * h.element_size() for h, _ in host)
    m2 = Model(wl, args.sparsity, dev, transposed=args.transposed)
    for _ in range(3):
        m2.sparsify(); m2.layers()
    if args.no_graph:
        replay = [(sparsify, layers), (m2.sparsify, m2.layers)]
    else:
        g2_sp, g2_ly = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2_sp):
            m2.sparsify()
        with torch.cuda.graph(g2_ly):
            m2.layers()
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

    ms_step, ms_sp, ms_gemm, ms_e2e = max_over_ranks([ms_step, ms_sp, ms_gemm, ms_e2e], dev)

    flops = step_flops(wl, m.n_attn, m.k_ffn)
    sbytes = sparsify_bytes(wl, 1.0 - args.sparsity, transposed=args.transposed)
    peaks = measured_peaks()
    n_gemm_launches = wl.n_layers * 8
    out = {
        "metric": METRIC, "value": job_throughput(world, flops, ms_step) / 1e9, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic (seeded N(0,sigma) tensors)",
        "config": {"workload": f"{wl.name}: {wl.n_layers} layers d_model={wl.d_m} heads={wl.n_heads}x{wl.d_h} "
                               f"ffn={wl.d_ffn} {wl.ffn} T={wl.tokens} sparsity={args.sparsity}"
                               + (" weights stored transposed" if args.transposed else ""),
                   "l2": "inputs larger than L2: 1.7 GB of weights/gradients per step, activations cycled over 4 sets",
                   "replicas": world, "launch": "eager" if args.no_graph else "cuda graph replay of the captured step"},
        "phases": {
            "sparsify": {"ms": ms_sp, "GB/s": sbytes / ms_sp / 1e6, "bytes": sbytes,
                         "frac_of_measured_hbm": sbytes / ms_sp / 1e6 / peaks["hbm_gbs"],
                         "frac_of_nominal_8TBs": sbytes / ms_sp / 1e6 / 8000.0},
            "gemm": {"ms": ms_gemm, "TFLOP/s": flops / ms_gemm / 1e9, "flops": flops,
                     "frac_of_nominal_2250": flops / ms_gemm / 1e9 / 2250.0},
        },
        "roofline": {"bound": "tensor", "kernel": "gemm_kernel", "achieved": flops / ms_gemm / 1e9,
                     "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": flops / ms_gemm / 1e9 / peaks["bf16_tflops_sustained"],
                     "traffic": NCU_GEMM_TRAFFIC_BYTES.get(wl.name) if (not args.layers and args.sparsity == 0.5 and not args.transposed) else None,
                     "traffic_unit": "bytes per launch (DRAM read + write, ncu)",
                     "peak_source": peaks["source"] + " (sustained cuBLAS bf16)",
                     "launches_per_step": n_gemm_launches, "avg_launch_ms": ms_gemm / n_gemm_launches},
        # the memory-bound part of the step against the measured copy bandwidth: score + select + compact as one unit
        # (sumsq_kernel and gather_kernel move all of its bytes; traffic = their DRAM bytes under ncu on 8 layers of
        # gpt2m, which grow in proportion to the layer count: 889.3 MB per 8 layers, profiles/sparsify_kernels_*.md)
        "roofline_hbm": {"bound": "hbm", "kernel": "sumsq_kernel + gather_kernel (+ finalize, select)",
                         "achieved": sbytes / ms_sp / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": sbytes / ms_sp / 1e6 / peaks["hbm_gbs"],
                         "traffic": (889.3e6 * wl.n_layers / 8 if (wl.name == "gpt2m" and args.sparsity == 0.5
                                                                   and not args.transposed) else None),
                         "traffic_unit": "bytes per step (DRAM read + write, ncu, scaled by layers)",
                         "peak_source": peaks["source"] + " (copy bandwidth)"},
        "e2e": {"value": job_throughput(world, flops, ms_e2e) / 1e9, "unit": "TFLOP/s", "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipeline": "two device copies of the model: the upload of step s+1 overlaps the compute of step s"},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_sample(wl, args.sparsity)
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# the CPU oracle on a bounded sample of the same step
# ---------------------------------------------------------------------------------------------

def cpu_sample(wl, sparsity: float, tokens: int = 256):
    """Layer 0 of the workload through the oracle: score + Fisher + select + compact at full size,
    then forward/backward of the compacted pairs on `tokens` token rows.  Returns the metric
    (algorithmic flops / wall time) for that sample."""
    import numpy as np
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
    t0 = time.perf_counter()
    groups = [("wq", "wk", None, "gq", "gk", None, 0, 0, wl.n_heads, wl.d_h, plan["qk"]),
              ("wv", "wo", None, "gv", "go", None, 0, 1, wl.n_heads, wl.d_h, plan["vo"]),
              ("w1", "w2", "w1b" if sw else None, "g1", "g2", "g1b" if sw else None, 0, 1, 1, wl.d_ffn, plan["ffn"])]
    c = {}
    for n1, n2, n1b, g1, g2, g1b, l1, l2, n_seg, seg_len, k in groups:
        _, ups = O.score_pair(w[n1], w[n2], l1, l2, n_seg, seg_len, w1b=w.get(n1b) if n1b else None)
        O.fisher_pair(g[g1], g[g2], l1, l2, n_seg, seg_len, float(wl.tokens), g1b=g.get(g1b) if g1b else None)
        kept = O.select_topk(ups.astype(np.float32), n_seg, seg_len, k)
        for nm, lay in ((n1, l1), (n2, l2), (n1b, l1), (g1, l1), (g2, l2), (g1b, l1)):
            if nm:
                src = w[nm] if nm in w else g[nm]
                c[nm] = O.compact(src, lay, kept, ld_out=pad8(len(kept), wl.elem_bytes) if lay == 0 else None)
    t1 = time.perf_counter()
    x = acts["x"]
    O.proj_fwd(x, c["wq"], 0, n_attn); O.proj_fwd(x, c["wk"], 0, n_attn); O.proj_fwd(x, c["wv"], 0, n_attn)
    O.outproj_fwd(acts["ctx"], c["wo"], 1, n_attn, wl.d_m)
    dX, _, _ = O.proj_bwd(x, c["wq"], 0, n_attn, acts["dq"])
    O.proj_bwd(x, c["wk"], 0, n_attn, acts["dk"], dX=dX)
    O.proj_bwd(x, c["wv"], 0, n_attn, acts["dv"])
    O.outproj_bwd(acts["ctx"], c["wo"], 1, n_attn, wl.d_m, acts["dout"])
    O.ffn_fwd(x, act, c["w1"], c["w2"], 0, 1, k_ffn, W1b=c.get("w1b"))
    O.ffn_bwd(x, act, c["w1"], c["w2"], 0, 1, k_ffn, acts["dy"], W1b=c.get("w1b"))
    t2 = time.perf_counter()
    flops = step_flops(wl, n_attn, k_ffn) / wl.n_layers * tokens / wl.tokens
    sbytes = sparsify_bytes(wl, 1.0 - sparsity) / wl.n_layers
    return {"value": flops / (t2 - t0) / 1e12, "unit": "TFLOP/s", "cores": 1, "kind": "oracle",
            "sample": f"layer 0 of {wl.name}: score+Fisher+select+compact at full size ({t1 - t0:.2f} s, "
                      f"{sbytes / (t1 - t0) / 1e9:.3f} GB/s), then fwd+bwd of the compacted QK/VO/FFN pairs on "
                      f"{tokens} of {wl.tokens} tokens ({t2 - t1:.2f} s)",
            "seconds": t2 - t0, "gemm_tflops": flops / (t2 - t1) / 1e12, "sparsify_GB/s": sbytes / (t1 - t0) / 1e9}


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
    plan = WL.kept_plan(wl, args.sparsity)
    flops = step_flops(wl, sum(plan["qk"]), plan["ffn"][0]) / wl.n_layers * tokens / wl.tokens
    v = flops / dt / 1e12
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
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="gpt2m")
    ap.add_argument("--sparsity", type=float, default=0.5)
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (small cases for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
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
