"""GPU parity, call by call through the C ABI: moe_route, moe_permute, weight packing,
moe_expert_ffn, moe_combine -- each against the CPU checker on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from synth import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


def shape(d, f, E=8, k=2, r=0, xd="bf16", bias="none", cfg_id=7):
    return W.LayerShape("t", cfg_id, d, f, n_experts=E, top_k=k, wd_rank=r, x_dtype=xd, bias=bias)


@pytest.mark.parametrize("sh,T,renorm", [
    (W.TINY, 16, True),
    (W.WEARABLE, 8, True),
    (W.PHONE, 257, True),                       # router bias, ragged last block
    (shape(512, 64, E=16, k=4), 33, True),
    (shape(264, 64, E=6, k=3), 19, True),       # E not a multiple of 8: scalar weight loads
    (shape(256, 64, E=64, k=8), 9, True),
    (shape(256, 64, E=8, k=8), 5, True),        # k = E
    (shape(256, 64, E=8, k=1), 5, True),        # k = 1: weight exactly 1
    (shape(256, 64, E=8, k=2, xd="f32"), 40, False),   # raw probabilities
])
def test_route_matches_checker(sh, T, renorm):
    lay, t, host = U.build(sh, T, renorm=renorm)
    idx, w, probs = lay.route(t["x"], want_probs=True)
    torch.cuda.synchronize()
    R, Wt, S, wo = O.route(host["x"], host["w_router"], host["b_router"], sh.top_k, renorm)
    ora = {"logits": R, "topk_idx": S, "topk_w": wo}
    U.check_routing(idx.cpu().numpy(), w.cpu().numpy(), ora, sh.top_k)
    assert np.allclose(probs.cpu().numpy(), Wt, atol=U.W_TOL, rtol=0)
    if sh.top_k == 1 and renorm:
        assert torch.all(w == 1.0)
    assert lay.check() == 0


def test_route_exact_ties_go_to_lower_index():
    sh = shape(256, 64, E=8, k=3)
    t = W.make_layer(sh, 4, device="cuda")
    t["w_router"].zero_()
    lay, t, host = U.build(sh, 4, tensors=t)
    idx, w, _ = lay.route(t["x"])
    assert idx.cpu().tolist() == [[0, 1, 2]] * 4
    assert torch.allclose(w, torch.full_like(w, 1 / 3), atol=1e-7)


@pytest.mark.parametrize("T,E,k", [(1, 8, 2), (16, 8, 2), (2048, 8, 2), (5000, 16, 4), (1025, 64, 8), (7, 6, 1)])
def test_permute_bit_exact(T, E, k):
    g = np.random.default_rng(T)
    S = np.stack([g.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    if T == 2048:
        S[:, 0] = 3                                  # one expert gets every token, others ragged
        S[:, 1] = np.where(S[:, 1] == 3, 4, S[:, 1])
    lay, _, _ = U.build(shape(256, 64, E=E, k=k), 1)
    offsets, perm, inv = lay.permute(torch.from_numpy(S).cuda())
    torch.cuda.synchronize()
    _, o_off, o_perm, o_inv = O.permute(S, E)
    assert np.array_equal(offsets.cpu().numpy(), o_off)
    assert np.array_equal(perm.cpu().numpy(), o_perm)
    assert np.array_equal(inv.cpu().numpy(), o_inv)
    assert lay.check() == 0


def test_pack_layouts():
    import paper_2503_00245_b200 as P
    sh = shape(72, 40, E=3)
    t = W.make_experts(sh, device="cuda")
    gud = P.pack_dense(t["w_gate"], t["w_up"], t["w_down"])
    assert torch.equal(gud[:, :, 0, :], t["w_gate"].transpose(1, 2))
    assert torch.equal(gud[:, :, 1, :], t["w_up"].transpose(1, 2))
    assert torch.equal(gud[:, :, 2, :], t["w_down"])
    t = W.make_experts(shape(72, 40, E=3, r=16), device="cuda")
    a, b, c, d = P.pack_wd(*(t[n] for n in ("gL", "gR", "uL", "uR", "dL", "dR")))
    assert torch.equal(a[:, :, 0, :], t["gL"].transpose(1, 2)) and torch.equal(a[:, :, 1, :], t["uL"].transpose(1, 2))
    assert torch.equal(b[:, :, 0, :], t["gR"].transpose(1, 2)) and torch.equal(b[:, :, 1, :], t["uR"].transpose(1, 2))
    assert torch.equal(c, t["dL"].transpose(1, 2)) and torch.equal(d, t["dR"].transpose(1, 2))


@pytest.mark.parametrize("sh,T,path", [
    (W.TINY, 16, 1), (W.TINY, 16, 2),
    (W.WEARABLE, 8, 1),
    (shape(136, 200, E=8, k=2), 5, 1),           # widths that are multiples of 8 only
    (shape(256, 512, E=8, k=2, r=32, xd="f32"), 16, 1),
    (shape(256, 512, E=8, k=2, r=32), 16, 2),
    (W.WEARABLE, 200, 2),
])
def test_expert_ffn_and_combine_match_checker(sh, T, path):
    lay, t, host = U.build(sh, T, path=path)
    ora = U.oracle_layer(host, sh.top_k)
    offsets = torch.from_numpy(ora["offsets"]).cuda()
    perm = torch.from_numpy(ora["perm"]).cuda()
    out = lay.expert_ffn(t["x"], offsets, perm)
    torch.cuda.synchronize()
    assert lay.check() == 0
    U.assert_close_rms(out.cpu().numpy().astype(np.float64), ora["out_slots"], what="out_slots")
    # combine on the checker's own slots (fp32-rounded) isolates the combine step
    o32 = torch.from_numpy(ora["out_slots"].astype(np.float32)).cuda()
    y = lay.combine(o32, torch.from_numpy(ora["topk_w"].astype(np.float32)).cuda(), torch.from_numpy(ora["inv"]).cuda())
    want = O.combine(o32.cpu().numpy().astype(np.float64), ora["topk_w"].astype(np.float32).astype(np.float64), ora["inv"])
    tol = 2.0 ** -8 if t["x"].dtype == torch.bfloat16 else 1e-6     # one rounding to the output type
    U.assert_close_rms(U.to64(y), want, tol=tol * 6, what="combine")
