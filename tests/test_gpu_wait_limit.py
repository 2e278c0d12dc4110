"""A device-side wait that runs out: the kernel must return by itself, report which wait gave up through
ecospa_device_status, leave the context usable, and the next ordinary call must be correct.

The wait is made to run out by shortening the limit to a microsecond on a product whose main loop lasts tens of
microseconds (the epilogue warps wait that long for the accumulator, the MMA issuer waits longer than that for the
first operand tiles): no barrier is removed and nothing is left unsignalled, the kernel only stops waiting early.
The product has a single 128-row tile, which the engine runs with one CTA per tile (no CTA pairs).
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_11641_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct():
    T, d_m, n = 128, 8192, 512
    g = torch.Generator().manual_seed(3)
    X = torch.randn((T, d_m), generator=g).to(torch.bfloat16)
    W = (torch.randn((d_m, n), generator=g) * 0.02).to(torch.bfloat16)
    Xd, Wd = X.to(DEV), W.to(DEV)
    Q = torch.zeros((T, n), dtype=torch.bfloat16, device=DEV)
    B.ecospa_device_status()                       # clean slate
    try:
        B.ecospa_set_device_wait_limit_ns(1000)
        B.ecospa_coupled_qk_fwd(Xd, Wd, None, n, Q, None)
        with pytest.raises(B.EcospaError) as ei:
            B.ecospa_device_status()
    finally:
        B.ecospa_set_device_wait_limit_ns(2_000_000_000)
    assert ei.value.status == 5                    # ECOSPA_ERR_TIMEOUT
    assert ei.value.code in (1, 2, 3, 4)
    assert B.ecospa_device_status() == 0           # the word was cleared by the read
    # the context is intact and the same call, with the ordinary limit, gives the right answer
    Q.zero_()
    B.ecospa_coupled_qk_fwd(Xd, Wd, None, n, Q, None)
    assert B.ecospa_device_status() == 0
    ref = O.proj_fwd(X, W, O.SHARED_COLS, n)
    got = Q.double().cpu().numpy()
    assert np.linalg.norm(got - ref) <= 2e-2 * np.linalg.norm(ref)
