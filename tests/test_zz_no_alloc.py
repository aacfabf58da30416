"""moe_layer_forward_static: the layer for callers that cannot allocate device memory (a plug-in in a host
application that owns all GPU memory, a real-time loop where cudaMalloc's device-wide synchronisation is
not allowed).  Its scratch is a __device__ array inside the library instead of cudaMalloc'ed memory.

Checked here through the C ABI against the ordinary entry point, moe_layer_forward, on two calls in a
row (the second call finds whatever the first left in the shared array), at one token and at several.
Collected last on purpose: if it fails, a run that stops at the first failure has run everything else.
"""
import pytest
import torch

from synth import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


def _pair(sh, T, step):
    """Output of the ordinary entry point and of the no-allocation one on the same fresh input."""
    from paper_2503_00245_b200 import binding as B
    lay, t, _ = U.build(sh, T, path=B.MOE_PATH_STREAM)
    x = W.make_x(sh, T, device="cuda", step=step)
    ref = lay.forward(x)
    torch.cuda.synchronize()
    assert lay.check() == 0
    y = torch.full_like(x, float("nan"))
    idx = torch.empty((T, sh.top_k), dtype=torch.int32, device="cuda")
    w = torch.empty((T, sh.top_k), dtype=torch.float32, device="cuda")
    return B, lay, x, ref, y, idx, w


E6 = W.LayerShape("six experts", 8, 136, 200, n_experts=6, top_k=3)


@pytest.mark.parametrize("sh,T", [
    (W.WEARABLE, 1), (W.WEARABLE, 8), (W.TINY, 16),
    (W.PHONE, 1),     # d_model at the limit
    (W.PHONE, 16),    # d_model and T at the limit: the accumulators fill the scratch array exactly
    (E6, 5),          # E not 8 or 16 with several tokens: the router runs as its own kernel first
])
def test_static_entry_matches_ordinary_entry_twice_in_a_row(sh, T):
    for step in (1, 2):                       # two calls in a row, different inputs
        B, lay, x, ref, y, idx, w = _pair(sh, T, step)
        rc = B.moe_layer_forward_static(lay.cfg, x, T, lay.weights, y, idx, w)
        assert rc == 0, rc
        torch.cuda.synchronize()
        assert B.moe_layer_forward_static(lay.cfg, x, 0, lay.weights, y) == 0      # nothing reported
        # same kernels, same fixed-point summation: the two entry points agree to the last bit, which is
        # well inside the layer's tolerance (max |diff| <= 2e-2 * RMS)
        a, b = y.float(), ref.float()
        assert torch.isfinite(a).all()
        assert float((a - b).abs().max()) <= U.Y_TOL * float(b.pow(2).mean().sqrt())
        assert torch.equal(y, ref)
        lay.close()


def test_static_entry_rejects_what_does_not_fit():
    from paper_2503_00245_b200 import binding as B
    lay, t, _ = U.build(W.TINY, 16, path=B.MOE_PATH_STREAM)
    y = torch.empty_like(t["x"])
    big_d = B.make_config(4096, 512, 8, 2)
    assert B.moe_layer_forward_static(big_d, t["x"], 1, lay.weights, y) == 2          # d_model > 2048
    assert B.moe_layer_forward_static(lay.cfg, t["x"], 17, lay.weights, y) == 2       # T > 16
    wd = B.make_config(256, 512, 8, 2, wd_rank=32)
    assert B.moe_layer_forward_static(wd, t["x"], 1, lay.weights, y) == 2             # decomposed experts
    assert B.moe_layer_forward_static(lay.cfg, t["x"], 16, lay.weights, y) == 1       # T > 1 without routing buffers
    lay.close()


def test_static_entry_single_token_without_routing_buffers_and_against_the_checker():
    """T == 1 with topk_idx / topk_w NULL, twice in a row; the second output also against the CPU checker."""
    from paper_2503_00245_b200 import binding as B
    sh = W.WEARABLE
    lay, t, host = U.build(sh, 1, path=B.MOE_PATH_STREAM)
    for step in (3, 4):
        x = W.make_x(sh, 1, device="cuda", step=step)
        ref = lay.forward(x)
        y = torch.full_like(x, float("nan"))
        assert B.moe_layer_forward_static(lay.cfg, x, 1, lay.weights, y) == 0
        torch.cuda.synchronize()
        assert B.moe_layer_forward_static(lay.cfg, x, 0, lay.weights, y) == 0
        assert torch.equal(y, ref)
    h = dict(host)
    h["x"] = W.to_host_bits(x)
    ora = U.oracle_layer(h, sh.top_k)
    if not O_near(ora, sh.top_k).any():
        U.assert_close_rms(U.to64(y), ora["y"])
    lay.close()


def O_near(ora, k):
    from oracle import moe_oracle as O
    return O.near_tie_tokens(ora["logits"], k, U.TIE_GAP)
