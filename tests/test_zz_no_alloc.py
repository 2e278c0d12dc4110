"""The allocation-free scoring entry point against the regular one.

Some users of this library cannot allocate device memory at the point where they need scores (they
run inside someone else's memory-managed region, or under a fixed memory budget), so they cannot
supply the workspace ecospa_score_pairs wants.  ecospa_score_pair_static keeps its scratch in a
fixed array inside the library instead.  This file checks, through the C ABI, that it returns what
the regular call returns -- on two calls in a row, because the array keeps the previous call's
contents -- and that it refuses pair groups whose scratch need is larger than the array.

Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import pytest
import torch

from paper_2511_11641_b200 import binding as B
from paper_2511_11641_b200 import block as BL
from paper_2511_11641_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda"
REL = 1e-5     # the tolerance of the score parity tests


def _regular(p, D, n_seg, n_samples):
    ups = torch.empty(D, dtype=torch.float32, device=DEV)
    raw = torch.empty(D, dtype=torch.float32, device=DEV)
    fis = torch.empty(n_seg, dtype=torch.float32, device=DEV)
    B.ecospa_score_pairs([p], n_samples, ups, raw, fis)
    torch.cuda.synchronize()
    return ups, raw, fis


def _static(p, D, n_seg, n_samples):
    ups = torch.full((D,), -3.0, dtype=torch.float32, device=DEV)
    raw = torch.full((D,), -3.0, dtype=torch.float32, device=DEV)
    fis = torch.full((n_seg,), -3.0, dtype=torch.float32, device=DEV)
    before = torch.cuda.memory_allocated()
    B.ecospa_score_pair_static(p, n_samples, ups, raw, fis)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    return ups, raw, fis


def _close(a, b):
    return torch.allclose(a, b, rtol=REL, atol=REL * float(b.abs().max()))


@pytest.mark.parametrize("name", ["llama1b", "gpt2m"])
def test_static_scratch_scores_match_regular_call_twice_in_a_row(name):
    wl = WL.WORKLOADS[name]
    dev_t = lambda d: {k: v.to(DEV) for k, v in d.items()}
    # two different layers back to back: the second call finds the first call's data in the array
    for layer in (0, 1):
        w, g = dev_t(WL.layer_weights(wl, layer)), dev_t(WL.layer_grads(wl, layer))
        pairs = BL.block_pairs(w, wl.n_heads, wl.d_h, wl.d_ffn, g)
        for p, D, n_seg in ((pairs[2], wl.d_ffn, 1), (pairs[0], wl.n_heads * wl.d_h, wl.n_heads)):
            ref = _regular(p, D, n_seg, float(wl.tokens))
            got = _static(p, D, n_seg, float(wl.tokens))
            for a, b in zip(got, ref):
                assert _close(a, b)
            got2 = _static(p, D, n_seg, float(wl.tokens))
            for a, b in zip(got2, got):
                assert torch.equal(a, b)


def test_static_scratch_rejects_oversized_pairs():
    limit = B.ecospa_score_pair_static_max_bytes()
    assert 0 < limit <= 16 << 20
    D, other = 320 * 1024, 512          # the stat/partial vectors of 320 Ki floats need more than 4 MiB
    w1 = torch.zeros((other, D), dtype=torch.bfloat16, device=DEV)
    w2 = torch.zeros((D, 8), dtype=torch.bfloat16, device=DEV)
    p = B.pair(B.PAIR_PLAIN, 1, D, w1, w2, B.SHARED_COLS, B.SHARED_ROWS)
    assert B.ecospa_score_workspace_bytes([p]) > limit
    ups = torch.full((D,), -3.0, dtype=torch.float32, device=DEV)
    with pytest.raises(B.EcospaError) as e:
        B.ecospa_score_pair_static(p, 1.0, ups)
    assert e.value.status == 3 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert torch.all(ups == -3.0)       # nothing was launched
