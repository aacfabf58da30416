"""GPU parity of moe_layer_forward against the CPU checker: the paper-shaped configurations and
the degenerate cases, streaming (decode) and tensor-core (prefill) paths."""
import numpy as np
import pytest
import torch

from synth import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu

STREAM, TENSOR = 1, 2


def shape(d, f, E=8, k=2, r=0, xd="bf16", bias="none", cfg_id=8):
    return W.LayerShape("t", cfg_id, d, f, n_experts=E, top_k=k, wd_rank=r, x_dtype=xd, bias=bias)


@pytest.mark.parametrize("sh,T,path", [
    (W.TINY, 16, STREAM),
    (W.TINY, 16, TENSOR),
    (W.WEARABLE, 1, 0),
    (W.WEARABLE, 8, 0),
    (W.WEARABLE, 512, 0),
    (W.PHONE, 1, 0),
    (W.PHONE, 2048, 0),                             # full-size prefill, uneven expert load (router bias)
    (W.PHONE_WD128, 2048, 0),
    (W.PHONE_WD1024, 2048, 0),
    (W.PHONE, 16, TENSOR),                          # tensor path with nearly empty 128-row tiles
    (shape(1440, 3840), 300, TENSOR),               # K not a multiple of 64, ragged groups
    (shape(136, 200, E=6, k=3), 37, TENSOR),        # tiny widths: K and N tails inside one tile
    (W.PHONE_WD128, 1, 0),
    (W.PHONE_WD1024, 1, 0),
    (W.PHONE_OFFLOAD, 1, 0),                        # E = 16, Zipf bias
    (shape(1440, 3840), 1, 0),                      # the paper's own phone-sized layer (Table 1 widths)
    (shape(432, 1280), 3, 0),                       # the paper's wearable-sized layer
    (shape(136, 200, E=6, k=3), 5, STREAM),
    (shape(256, 512, k=1), 4, STREAM),
    (shape(256, 512, k=8), 2, STREAM),
    (shape(256, 512, r=64), 16, STREAM),
    (shape(256, 512, r=64, xd="f32"), 7, STREAM),
    # several tokens through the streaming kernel: every instantiation of the tensor-core pass
    (W.PHONE, 8, STREAM),                           # d > 1024, bf16 rows
    (shape(2048, 1024, xd="f32"), 5, STREAM),       # d > 1024, fp32 rows (head + remainder)
    (shape(1440, 3840), 9, STREAM),                 # d not a multiple of 32 x 8: ragged k groups and column blocks
    (W.PHONE_OFFLOAD, 16, STREAM),                  # E = 16 routed inside the kernel, experts with more than 8 tokens
    (shape(256, 512, E=64, k=8), 4, STREAM),        # E = 64: router as its own kernel, many active experts
    # the paper's ablation grid (Fig. 7): active experts 1..8 of 8, total experts 2..16 with 2 active
    (shape(256, 512, E=8, k=4), 1, 0),
    (shape(256, 512, E=8, k=8), 1, 0),
    (shape(256, 512, E=2, k=2), 1, 0),
    (shape(256, 512, E=4, k=2), 3, 0),
    (shape(256, 512, E=16, k=2), 6, 0),
    (shape(256, 512, E=2, k=1), 40, 0),             # tensor path with two experts
    # the paper's weight-decomposed layers (Table 1: hidden 1600 / 400, rank = half the hidden width, Section 2.2)
    (shape(1600, 4352, r=800), 1, 0),               # streaming kernel at the paper's phone-WD widths
    (shape(1600, 4352, r=800), 300, 0),             # tensor path, rank not a multiple of 64
    (shape(400, 1280, r=200), 1, 0),                # wearable-WD widths
    (shape(400, 1280, r=200), 64, 0),
    (shape(4096, 512), 4, 0),                       # dense, d_model beyond the streaming kernel: tensor path at small T
    # one token, accumulator words that count their arrivals: CTAs without a share (fewer hidden units than CTAs per
    # expert) still have to be counted; one and eight choices change the arrivals a word waits for; fp32 rows
    (shape(256, 64), 1, 0),
    (shape(256, 40, E=8, k=1), 1, 0),
    (shape(1024, 2816, E=8, k=8), 1, 0),
    (shape(2048, 1024, E=8, k=1, xd="f32"), 1, 0),
    (shape(256, 512, E=64, k=4), 1, 0),             # two logits per lane in the routing warp
])
def test_layer_forward_matches_checker(sh, T, path):
    lay, t, host = U.build(sh, T, path=path)
    rel, _, _ = U.check_layer(lay, t, host, sh.top_k)
    assert rel <= U.Y_TOL


@pytest.mark.parametrize("sh,T", [(shape(1600, 4352, r=800), 2048), (W.PHONE, 2048), (W.PHONE_WD1024, 2048)])
def test_full_prefill_error_beyond_output_rounding(sh, T):
    """Full-size prefill, 3 to 4 million bf16 outputs.  There the rounding of y to bf16 alone comes to 1.7e-2 * RMS
    and more at the largest outputs, so this test bounds what the kernels add to it: every element within half a
    bf16 ulp of the checker's value plus 1e-2 * RMS (six standard deviations of what rounding the hidden activations to bf16 leaves in y)."""
    lay, t, host = U.build(sh, T)
    _, ora, y = U.check_layer(lay, t, host, sh.top_k, tol=1.0)
    U.assert_close_in_output_type(U.to64(y), ora["y"])


def test_all_tokens_to_one_expert_stream():
    """Bias forces experts 5 and 2 into every token's set: each serves 16 tokens (two passes of 8),
    the other experts get nothing."""
    sh = shape(256, 512)
    t = W.make_layer(sh, 16, device="cuda")
    b = torch.zeros(8, device="cuda")
    b[5] = 50.0
    b[2] = 40.0
    t["b_router"] = b
    lay, t, host = U.build(sh, 16, path=STREAM, tensors=t)
    rel, ora, _ = U.check_layer(lay, t, host, 2)
    assert ora["counts"].tolist() == [0, 0, 16, 0, 0, 16, 0, 0]


@pytest.mark.parametrize("sh,T", [
    (W.WEARABLE, 8),                       # fused streaming kernel against the four calls (streaming FFN per slot)
    (W.PHONE, 1),                          # one launch with dynamic stage hand-out against the four calls
    (shape(1440, 3840), 300),              # tensor path: layer (route, permute, gather, two GEMMs, combine) against the calls
    (W.PHONE_WD1024, 1),                   # streamed factor products in one launch against the four-phase per-slot kernel
    (shape(256, 512, r=64, xd="f32"), 7),
])
def test_layer_equals_composition_of_steps(sh, T):
    lay, t, host = U.build(sh, T)
    y = lay.forward(t["x"])
    idx, w, _ = lay.route(t["x"])
    offsets, perm, inv = lay.permute(idx)
    out = lay.expert_ffn(t["x"], offsets, perm)
    y2 = lay.combine(out, w, inv)
    torch.cuda.synchronize()
    assert lay.check() == 0
    a, b = y.float(), y2.float()
    assert torch.max(torch.abs(a - b)) <= 2.0 ** -7 * torch.sqrt(torch.mean(b * b))   # one bf16 ulp of slack


def test_repeat_calls_are_bitwise_identical():
    lay, t, _ = U.build(W.WEARABLE, 8)
    y1 = lay.forward(t["x"]).clone()
    y2 = lay.forward(t["x"]).clone()
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)


@pytest.mark.parametrize("T", [1, 8, 16])
def test_back_to_back_calls_with_different_inputs(T):
    """Calls queued without a host sync in between, each with its own x: a call must not see anything (token
    rows, routing, partial sums) a neighbouring call left in shared memory or in the accumulators."""
    sh = W.WEARABLE
    lay, t, host = U.build(sh, T, path=STREAM)
    xs = [W.make_x(sh, T, device="cuda", step=s) for s in range(4)]
    ys = [lay.forward(x).clone() for x in xs]
    torch.cuda.synchronize()
    assert lay.check() == 0
    for x, y in zip(xs, ys):
        h = dict(host)
        h["x"] = W.to_host_bits(x)
        ora = U.oracle_layer(h, sh.top_k)
        tie = O_near(ora, sh.top_k)
        if tie.any():
            continue            # the selection itself is undecided for some token: covered by check_layer elsewhere
        U.assert_close_rms(U.to64(y), ora["y"])


@pytest.mark.parametrize("sh,T", [(W.WEARABLE, 1), (W.WEARABLE, 8), (W.PHONE, 1), (W.PHONE_WD128, 1), (W.PHONE_WD1024, 1)])
def test_long_run_of_queued_calls_is_bitwise_stable(sh, T):
    """Two thousand launches queued back to back, alternating four inputs, each output kept: every output must
    equal, bit for bit, the first one its input produced.  The fixed-point partial sums, the arrival counter that
    runs over launches and the finalisers' reads are ordered only by release/acquire operations; a launch that
    finalised before a neighbour's (or its own) sums had landed would show here."""
    lay, t, host = U.build(sh, T, path=STREAM)
    xs = [W.make_x(sh, T, device="cuda", step=s) for s in range(4)]
    first = [lay.forward(x).clone() for x in xs]
    torch.cuda.synchronize()
    n = 2000
    out = torch.empty((n,) + tuple(first[0].shape), dtype=first[0].dtype, device="cuda")
    for i in range(n):
        lay.forward(xs[i % 4], y=out[i])
    torch.cuda.synchronize()
    assert lay.check() == 0
    for j in range(4):
        same = (out[j::4].view(torch.int16 if out.dtype == torch.bfloat16 else torch.int32)
                == first[j].view(torch.int16 if out.dtype == torch.bfloat16 else torch.int32))
        assert bool(same.all()), f"input {j}: {int((~same).sum())} differing elements over {n // 4} launches"


def O_near(ora, k):
    from oracle import moe_oracle as O
    return O.near_tie_tokens(ora["logits"], k, U.TIE_GAP)


def test_argument_errors_are_reported_not_run():
    from paper_2503_00245_b200 import binding as B
    lay, t, _ = U.build(W.TINY, 16)
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    y = torch.empty_like(t["x"])
    with pytest.raises(B.MoeError) as e:
        B.moe_layer_forward(lay.ctx, t["x"], 16, lay.weights, y, ws=small)
    assert e.value.status == 3
    lay2, t2, _ = U.build(W.TINY, 32, path=STREAM, max_tokens=32)
    with pytest.raises(B.MoeError) as e:
        lay2.forward(t2["x"])
    assert e.value.status == 2                      # streaming path is limited to 16 tokens
    B.moe_layer_forward(lay.ctx, t["x"], 0, lay.weights, y, ws=lay.ws)   # T = 0: no-op
    assert lay.check() == 0


def _decode_us(sh, reps=200):
    """Median-free, simple timing of batch-1 decode over a ring of distinct layers (weights beyond L2 are not
    needed for a comparison between shapes: every shape is timed the same way)."""
    lays = [U.build(sh, 1, layer=l)[0] for l in range(6)]
    x = W.make_x(sh, 1, device="cuda")
    ys = [torch.empty_like(x) for _ in lays]
    for _ in range(3):
        for lay, y in zip(lays, ys):
            lay.forward(x, y=y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        for lay, y in zip(lays, ys):
            lay.forward(x, y=y)
    e1.record()
    torch.cuda.synchronize()
    for lay in lays:
        assert lay.check() == 0
        lay.close()
    return e0.elapsed_time(e1) * 1e3 / (reps * len(lays))


def test_decode_time_follows_active_not_total_experts():
    """The paper's ablation (Section 3.4.4, Fig. 7): generation speed falls with the number of ACTIVE experts and
    does not depend on the TOTAL number, because only the selected experts' weights are touched.  Wearable widths,
    batch-1 decode; generous bounds (a launch has a fixed cost besides the weight stream)."""
    base = W.WEARABLE
    t_k1 = _decode_us(base.with_(top_k=1))
    t_k8 = _decode_us(base.with_(top_k=8))
    t_e2 = _decode_us(base.with_(n_experts=2))
    t_e16 = _decode_us(base.with_(n_experts=16))
    assert t_k8 > 2.0 * t_k1, (t_k1, t_k8)
    assert abs(t_e16 - t_e2) < 0.2 * max(t_e16, t_e2), (t_e2, t_e16)


@pytest.mark.parametrize("sh,T", [(W.WEARABLE, 1), (W.PHONE, 1), (W.TINY, 16), (W.WEARABLE, 8)])
def test_streaming_path_writes_y_to_mapped_host_memory(sh, T):
    """On the streaming path y may be mapped pinned host memory: the finalising CTAs store it themselves."""
    lay, t, _ = U.build(sh, T, path=STREAM)
    for step in range(2):
        x = W.make_x(sh, T, device="cuda", step=step)
        ref = lay.forward(x)
        hy = torch.zeros((T, sh.d_model), dtype=x.dtype).pin_memory()
        lay.forward(x, y=hy)
        torch.cuda.synchronize()
        assert lay.check() == 0
        assert torch.equal(hy, ref.cpu())
    lay.close()


@pytest.mark.parametrize("sh", [W.WEARABLE, W.PHONE])
def test_one_ctx_alternating_token_counts(sh):
    """One ctx, calls with one token and with several in turn: the two ways of finishing the sums (words that count
    their arrivals; the arrival counter) share the accumulators, and each must leave them zero for the other.  Every
    call's output equals that of a fresh ctx given the same rows."""
    lay, t, _ = U.build(sh, 8, path=STREAM)
    x8 = t["x"]
    fresh1, _, _ = U.build(sh, 1, path=STREAM, tensors=t)
    fresh8, _, _ = U.build(sh, 8, path=STREAM, tensors=t)
    want8 = fresh8.forward(x8).clone()
    want1 = [fresh1.forward(x8[i:i + 1]).clone() for i in range(3)]
    torch.cuda.synchronize()
    for rep in range(3):
        for i in range(3):
            assert torch.equal(lay.forward(x8[i:i + 1]), want1[i])
            assert torch.equal(lay.forward(x8), want8)
    torch.cuda.synchronize()
    assert lay.check() == 0 and fresh1.check() == 0 and fresh8.check() == 0
    for l in (lay, fresh1, fresh8):
        l.close()
