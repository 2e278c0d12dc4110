"""Buffer plumbing for the compacted-pair forward/backward calls (allocation and argument order only)."""
from __future__ import annotations

from typing import Dict

import torch

from . import binding as B
from .block import pad8


def ffn_buffers(T: int, d_m: int, k: int, act: int, dtype: torch.dtype, device, transposed: bool = False) -> Dict[str, torch.Tensor]:
    """Outputs and saved tensors of one FFN forward+backward (H, Hb, A are always bf16).  transposed: weights are
    stored the other way round (W_1 as k x d_m, W_2 as d_m x k), and so are their gradients."""
    kp = pad8(k, 2)
    kpw = pad8(k, 2 if dtype == torch.bfloat16 else 4)
    sw = act == B.ACT_SWIGLU
    d = {
        "Y": torch.empty((T, d_m), dtype=dtype, device=device),
        "H": torch.empty((T, kp), dtype=torch.bfloat16, device=device),
        "A": torch.empty((T, kp), dtype=torch.bfloat16, device=device),
        "dX": torch.empty((T, d_m), dtype=dtype, device=device),
        "dW1": torch.zeros((k, d_m) if transposed else (d_m, kpw), dtype=dtype, device=device),
        "dW2": torch.zeros((d_m, kpw) if transposed else (k, d_m), dtype=dtype, device=device),
        "db2": torch.empty((d_m,), dtype=dtype, device=device),
    }
    if sw:
        d["Hb"] = torch.empty((T, kp), dtype=torch.bfloat16, device=device)
        d["dW1b"] = torch.zeros((k, d_m) if transposed else (d_m, kpw), dtype=dtype, device=device)
    else:
        d["db1"] = torch.empty((k,), dtype=dtype, device=device)
    code = B.F32 if dtype == torch.float32 else B.BF16
    d["ws"] = torch.empty(max(16, B.ecospa_ffn_workspace_bytes(T, d_m, k, act, code)), dtype=torch.uint8, device=device)
    return d


def ffn_fwd_bwd(X, dY, act: int, w1c, w2c, k: int, buf: Dict[str, torch.Tensor], w1bc=None, b1c=None, b2=None,
                bias_grads: bool = True, **layouts) -> None:
    """bias_grads=False: the layer has no biases, so db1 / db2 (column sums of dH / dY) are not asked for."""
    B.ecospa_coupled_ffn_fwd(X, act, w1c, w2c, k, buf["Y"], buf["H"], buf["A"], w1b_c=w1bc, Hb=buf.get("Hb"),
                             b1_c=b1c, b2=b2, workspace=buf["ws"], **layouts)
    B.ecospa_coupled_ffn_bwd(X, act, w1c, w2c, k, buf["H"], buf["A"], dY, buf["dX"], buf["dW1"], buf["dW2"],
                             w1b_c=w1bc, Hb=buf.get("Hb"), dW1b_c=buf.get("dW1b"), db1_c=buf.get("db1") if bias_grads else None,
                             db2=buf["db2"] if bias_grads else None, workspace=buf["ws"], **layouts)
