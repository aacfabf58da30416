"""Pins for the CPU checker: closed forms, hand-worked values, invariants, library
special cases and brute force, so that a dropped term, wrong sign, wrong index or
transposed operand in oracle/ fails here.  No GPU involved."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from synth import workloads as W

F64 = torch.float64


def rand_layer(seed, T, d, f, E, wd_rank=0):
    shape = W.LayerShape("t", 9, d, f, n_experts=E, wd_rank=wd_rank, x_dtype="f32")
    L = W.make_layer(shape, T, layer=seed)
    return {k: W.to_host_bits(v) for k, v in L.items()}


def experts_of(L):
    return {k: v for k, v in L.items() if k not in ("x", "w_router", "b_router")}


# ------------------------------------------------------------------ widening
def test_widen_known_bf16_patterns():
    bits = np.array([0x3F80, 0xC000, 0x0000, 0x8000, 0x3DCC, 0x7F7F, 0x0080], dtype=np.uint16)
    want = [1.0, -2.0, 0.0, -0.0, 0.099609375, 3.3895313892515355e38, 2.0 ** -126]
    got = O.widen(bits)
    assert got.dtype == np.float64
    assert got.tolist() == want
    assert math.copysign(1.0, got[3]) == -1.0


def test_widen_matches_torch_bf16_conversion():
    t = torch.randn(4096, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    assert np.array_equal(O.widen(W.to_host_bits(t)), t.to(F64).numpy())
    x32 = np.float32([0.1, -3.25e-7])
    assert np.array_equal(O.widen(x32), x32.astype(np.float64))


# ------------------------------------------------------------------ router
def test_router_logits_hand_example_and_orientation():
    # x is [T=1, d=3], W_r is [d=3, E=2]: a transposed operand cannot even multiply,
    # and the numbers below are worked by hand.
    x = np.float64([[1.0, 2.0, -1.0]])
    Wr = np.float64([[1.0, 0.5], [0.25, -1.0], [2.0, 4.0]])
    R = O.router_logits(x, Wr, np.float64([10.0, 20.0]))
    assert R.tolist() == [[1.0 + 0.5 - 2.0 + 10.0, 0.5 - 2.0 - 4.0 + 20.0]]
    assert O.router_logits(x, Wr).tolist() == [[-0.5, -5.5]]


def test_softmax_closed_forms_and_library():
    R = np.float64([[0.0, math.log(3.0)], [5.0, 5.0], [1000.0, 0.0]])
    Wt = O.softmax(R)
    assert np.allclose(Wt[0], [0.25, 0.75], rtol=0, atol=1e-15)
    assert Wt[1].tolist() == [0.5, 0.5]
    assert Wt[2].tolist() == [1.0, 0.0]            # max-subtraction: no overflow
    g = np.random.default_rng(0).normal(size=(64, 16)) * 3
    assert np.allclose(O.softmax(g), torch.softmax(torch.from_numpy(g), dim=1).numpy(), rtol=1e-14, atol=0)
    assert np.allclose(O.softmax(g + 7.25), O.softmax(g), rtol=1e-13, atol=0)   # shift invariance
    assert np.allclose(O.softmax(g).sum(1), 1.0, rtol=0, atol=1e-15)


def test_top_k_order_ties_and_library():
    Wt = np.float64([[0.1, 0.4, 0.4, 0.1], [0.25, 0.25, 0.25, 0.25], [0.0, 0.1, 0.2, 0.7]])
    assert O.top_k(Wt, 2).tolist() == [[1, 2], [0, 1], [3, 2]]
    assert O.top_k(Wt, 3).tolist() == [[1, 2, 0], [0, 1, 2], [3, 2, 1]]
    g = np.random.default_rng(1).random((200, 8))
    ref = torch.topk(torch.from_numpy(g), 3, dim=1).indices.numpy()
    assert np.array_equal(O.top_k(g, 3), ref)
    assert O.top_k(g, 3).dtype == np.int32


def test_gate_weights_identities():
    L = rand_layer(3, 33, 64, 32, 8)
    R, Wt, S, w = O.route(L["x"], L["w_router"], None, 2, True)
    assert np.allclose(w.sum(1), 1.0, atol=1e-15)
    assert np.all(w[:, 0] >= w[:, 1])
    # softmax -> top-k -> renormalise equals a softmax over the selected logits alone
    sel = np.take_along_axis(R, S.astype(np.int64), 1)
    assert np.allclose(w, O.softmax(sel), rtol=1e-13, atol=0)
    # without renormalisation the weights are the raw probabilities
    _, _, S2, w2 = O.route(L["x"], L["w_router"], None, 2, False)
    assert np.array_equal(S2, S)
    assert np.array_equal(w2, np.take_along_axis(Wt, S.astype(np.int64), 1))
    assert np.all(w2.sum(1) < 1.0)


def test_route_degenerate_cases():
    x = rand_layer(4, 5, 16, 8, 8)["x"]
    zero = np.zeros((16, 8), dtype=np.float32)
    _, Wt, S, w = O.route(x, zero, None, 3, True)
    assert S.tolist() == [[0, 1, 2]] * 5                      # all tied: lowest indices win
    assert np.allclose(w, 1.0 / 3.0, atol=1e-16) and np.allclose(Wt, 0.125)
    bias = np.zeros(8, dtype=np.float32)
    bias[5] = 50.0
    L = rand_layer(5, 9, 16, 8, 8)
    _, _, S, w = O.route(L["x"], L["w_router"], bias, 2, True)
    assert np.all(S[:, 0] == 5) and np.all(w[:, 0] > 0.999999)
    # k = E: every expert selected, weights are the full softmax
    _, Wt, S, w = O.route(L["x"], L["w_router"], None, 8, True)
    assert np.array_equal(np.sort(S, 1), np.tile(np.arange(8), (9, 1)))
    assert np.allclose(np.take_along_axis(w, np.argsort(S, 1), 1), Wt, rtol=1e-14)


def test_near_tie_detector():
    R = np.float64([[3.0, 2.0, 1.99995, 0.0], [3.0, 2.0, 1.9, 0.0]])
    assert O.near_tie_tokens(R, 2).tolist() == [True, False]
    assert O.near_tie_tokens(R, 1).tolist() == [False, False]
    assert O.near_tie_tokens(R, 4).tolist() == [False, False]


# ------------------------------------------------------------------ permutation
def test_permute_hand_example():
    S = np.int32([[2, 0], [0, 1], [2, 1]])          # pairs p: 0:(e2) 1:(e0) 2:(e0) 3:(e1) 4:(e2) 5:(e1)
    counts, offsets, perm, inv = O.permute(S, 4)
    assert counts.tolist() == [2, 2, 2, 0]
    assert offsets.tolist() == [0, 2, 4, 6, 6]
    assert perm.tolist() == [1, 2, 3, 5, 0, 4]
    assert inv.tolist() == [4, 0, 1, 2, 5, 3]


def test_permute_structure_and_library_sort():
    g = np.random.default_rng(2)
    for T, E, k in [(1, 8, 2), (37, 8, 2), (64, 16, 4), (5, 4, 4)]:
        S = np.stack([g.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
        counts, offsets, perm, inv = O.permute(S, E)
        assert offsets[0] == 0 and offsets[E] == T * k and counts.sum() == T * k
        assert np.array_equal(perm[inv], np.arange(T * k)) and np.array_equal(inv[perm], np.arange(T * k))
        assert np.array_equal(perm, np.argsort(S.reshape(-1), kind="stable"))   # stable sort by expert
        for e in range(E):
            seg = perm[offsets[e]:offsets[e + 1]]
            assert np.all(S.reshape(-1)[seg] == e) and np.all(np.diff(seg) > 0)


# ------------------------------------------------------------------ experts
def test_silu_closed_form_and_library():
    z = np.float64([0.0, math.log(3.0), -math.log(3.0), 40.0, -40.0])
    s = O.silu(z)
    assert s[0] == 0.0
    assert abs(s[1] - 0.75 * math.log(3.0)) < 1e-15
    assert abs(s[2] + 0.25 * math.log(3.0)) < 1e-15
    assert abs(s[3] - 40.0) < 1e-12 and abs(s[4]) < 1e-15
    g = np.random.default_rng(3).normal(size=1000) * 4
    assert np.allclose(s := O.silu(g), torch.nn.functional.silu(torch.from_numpy(g)).numpy(), rtol=1e-14, atol=1e-300)


def hand_layer():
    ln3 = math.log(3.0)
    x = np.float64([[1.0, 2.0]])
    Wr = np.float64([[1.0, 0.0], [0.0, 1.0]])                 # logits = x = [1, 2]
    Wg = np.float64([[[0.0, 0.0], [0.0, 0.0]], [[ln3, 0.0], [0.0, 0.0]]])   # expert 1: g = [ln3, 0]
    Wu = np.float64([[[1.0, 1.0], [1.0, 1.0]], [[2.0, 5.0], [1.0, 1.0]]])   # expert 1: u = [4, 7]; expert 0: u = [3, 3]
    Wd = np.float64([[[1.0, 2.0], [3.0, 4.0]], [[1.0, -1.0], [9.0, 9.0]]])
    return x, Wr, {"w_gate": Wg, "w_up": Wu, "w_down": Wd}


def test_layer_hand_worked_top1():
    x, Wr, ex = hand_layer()
    out = O.layer_forward(x, Wr, None, ex, k=1)
    ln3 = math.log(3.0)
    assert out["topk_idx"].tolist() == [[1]] and out["topk_w"].tolist() == [[1.0]]
    # h = silu([ln3, 0]) * [4, 7] = [3 ln3, 0];  o = h @ [[1,-1],[9,9]] = [3 ln3, -3 ln3]
    assert np.allclose(out["y"], [[3 * ln3, -3 * ln3]], rtol=1e-15)


def test_layer_hand_worked_top2_no_renorm_and_renorm():
    x, Wr, ex = hand_layer()
    ln3 = math.log(3.0)
    # expert 0 has a zero gate matrix -> silu(0) = 0 -> contributes nothing
    p1 = math.e / (1.0 + math.e)
    out = O.layer_forward(x, Wr, None, ex, k=2, renorm=False)
    assert out["topk_idx"].tolist() == [[1, 0]]
    assert np.allclose(out["topk_w"], [[p1, 1 - p1]], rtol=1e-15)
    assert np.allclose(out["y"], [[p1 * 3 * ln3, -p1 * 3 * ln3]], rtol=1e-14)
    # make expert 0 count: gate row so that g0 = [ln3, ln3], u0 = [3, 3] -> h0 = 2.25 ln3 [1, 1]
    ex["w_gate"][0] = np.float64([[ln3, ln3], [0.0, 0.0]])
    out = O.layer_forward(x, Wr, None, ex, k=2, renorm=True)
    o0 = 2.25 * ln3 * np.float64([1.0 + 3.0, 2.0 + 4.0])
    o1 = np.float64([3 * ln3, -3 * ln3])
    assert np.allclose(out["y"][0], p1 * o1 + (1 - p1) * o0, rtol=1e-14)
    assert np.allclose(out["out_slots"][out["inv"][0]], o1, rtol=1e-15)   # pair (t0, j0) = expert 1


def torch_swiglu(x, Wg, Wu, Wd):
    g, u = x @ Wg, x @ Wu
    return (torch.nn.functional.silu(g) * u) @ Wd


def test_k_equals_E_is_dense_softmax_mixture():
    L = rand_layer(6, 7, 48, 40, 4)
    out = O.layer_forward(L["x"], L["w_router"], None, experts_of(L), k=4)
    x = torch.from_numpy(O.widen(L["x"]))
    P = torch.softmax(x @ torch.from_numpy(O.widen(L["w_router"])), dim=1)
    y = torch.zeros(7, 48, dtype=F64)
    for e in range(4):      # every expert for every token, mixed by the full softmax
        y += P[:, e:e + 1] * torch_swiglu(x, *(torch.from_numpy(O.widen(L[n][e])) for n in ("w_gate", "w_up", "w_down")))
    assert np.allclose(out["y"], y.numpy(), rtol=1e-12, atol=1e-13)


def test_top1_is_single_dense_swiglu():
    L = rand_layer(7, 9, 32, 24, 8)
    out = O.layer_forward(L["x"], L["w_router"], None, experts_of(L), k=1)
    assert np.all(out["topk_w"] == 1.0)
    x = torch.from_numpy(O.widen(L["x"]))
    am = torch.argmax(x @ torch.from_numpy(O.widen(L["w_router"])), dim=1)
    for t in range(9):
        e = int(am[t])
        assert out["topk_idx"][t, 0] == e
        ref = torch_swiglu(x[t:t + 1], *(torch.from_numpy(O.widen(L[n][e])) for n in ("w_gate", "w_up", "w_down")))
        assert np.allclose(out["y"][t], ref[0].numpy(), rtol=1e-12, atol=1e-14)


def test_brute_force_python_loops_tiny():
    L = rand_layer(8, 3, 8, 8, 4)
    k = 2
    out = O.layer_forward(L["x"], L["w_router"], None, experts_of(L), k=k)
    x, Wr = O.widen(L["x"]), O.widen(L["w_router"])
    Wg, Wu, Wd = (O.widen(L[n]) for n in ("w_gate", "w_up", "w_down"))
    T, d = x.shape
    E, _, f = Wg.shape
    for t in range(T):
        logit = [sum(x[t][i] * Wr[i][e] for i in range(d)) for e in range(E)]
        m = max(logit)
        p = [math.exp(v - m) for v in logit]
        p = [v / sum(p) for v in p]
        chosen = sorted(range(E), key=lambda e: (-p[e], e))[:k]
        mask = [1.0 if e in chosen else 0.0 for e in range(E)]
        norm = sum(p[e] * mask[e] for e in range(E))
        y = [0.0] * d
        for e in range(E):                  # evaluate every expert, mask afterwards
            g = [sum(x[t][i] * Wg[e][i][c] for i in range(d)) for c in range(f)]
            u = [sum(x[t][i] * Wu[e][i][c] for i in range(d)) for c in range(f)]
            h = [g[c] / (1.0 + math.exp(-g[c])) * u[c] for c in range(f)]
            for n in range(d):
                y[n] += mask[e] * p[e] / norm * sum(h[c] * Wd[e][c][n] for c in range(f))
        assert out["topk_idx"][t].tolist() == chosen
        assert np.allclose(out["y"][t], y, rtol=1e-12, atol=1e-14)


def test_one_hot_input_reads_single_rows():
    L = rand_layer(9, 1, 16, 12, 4)
    Wg, Wu, Wd = (O.widen(L[n]) for n in ("w_gate", "w_up", "w_down"))
    x = np.zeros((1, 16), dtype=np.float32)
    x[0, 5] = 1.0
    _, offsets, perm, _ = O.permute(np.int32([[2]]), 4)
    o = O.expert_ffn_dense(x, L["w_gate"], L["w_up"], L["w_down"], offsets, perm, 1)
    g, u = Wg[2][5], Wu[2][5]                         # row 5 of expert 2's matrices
    assert np.allclose(o[0], (g / (1 + np.exp(-g)) * u) @ Wd[2], rtol=1e-13)


def test_wd_factored_equals_reconstructed():
    L = rand_layer(10, 6, 32, 40, 4, wd_rank=8)
    out = O.layer_forward(L["x"], L["w_router"], None, experts_of(L), k=2)
    x = O.widen(L["x"])
    f = {n: O.widen(L[n]) for n in ("gL", "gR", "uL", "uR", "dL", "dR")}
    assert O.reconstruct(L["gL"][1], L["gR"][1]).shape == (32, 40)
    assert O.reconstruct(L["dL"][1], L["dR"][1]).shape == (40, 32)
    for s, p in enumerate(out["perm"]):
        t, e = p // 2, out["topk_idx"].reshape(-1)[p]
        g = (x[t] @ f["gL"][e]) @ f["gR"][e]           # factored order: (x L) R
        u = (x[t] @ f["uL"][e]) @ f["uR"][e]
        h = g / (1 + np.exp(-g)) * u
        o = (h @ f["dL"][e]) @ f["dR"][e]
        assert np.allclose(out["out_slots"][s], o, rtol=1e-10, atol=1e-13)
    # and the dense path fed the reconstructed matrices gives the same layer output
    dense = {"w_gate": np.stack([f["gL"][e] @ f["gR"][e] for e in range(4)]),
             "w_up": np.stack([f["uL"][e] @ f["uR"][e] for e in range(4)]),
             "w_down": np.stack([f["dL"][e] @ f["dR"][e] for e in range(4)])}
    out2 = O.layer_forward(L["x"], L["w_router"], None, dense, k=2)
    assert np.array_equal(out2["y"], out["y"])


def test_token_permutation_invariance():
    L = rand_layer(11, 12, 32, 24, 8)
    out = O.layer_forward(L["x"], L["w_router"], None, experts_of(L), k=2)
    p = np.random.default_rng(5).permutation(12)
    out_p = O.layer_forward(L["x"][p], L["w_router"], None, experts_of(L), k=2)
    assert np.array_equal(out_p["topk_idx"], out["topk_idx"][p])
    assert np.allclose(out_p["topk_w"], out["topk_w"][p], rtol=1e-15)
    assert np.allclose(out_p["y"], out["y"][p], rtol=1e-12, atol=1e-15)


def test_combine_hand_example():
    o = np.float64([[1.0, 10.0], [2.0, 20.0], [3.0, 30.0], [4.0, 40.0]])
    w = np.float64([[0.5, 0.5], [0.25, 0.75]])
    inv = np.int32([2, 0, 1, 3])        # pair (t0,j0)->slot 2, (t0,j1)->0, (t1,j0)->1, (t1,j1)->3
    y = O.combine(o, w, inv)
    assert y.tolist() == [[0.5 * 3 + 0.5 * 1, 0.5 * 30 + 0.5 * 10], [0.25 * 2 + 0.75 * 4, 0.25 * 20 + 0.75 * 40]]


def test_forced_routing_and_empty_experts():
    L = rand_layer(12, 4, 16, 8, 8)
    forced = np.int32([[7, 7 - 1]] * 4)              # experts 0..5 receive nothing
    out = O.layer_forward(L["x"], L["w_router"], None, experts_of(L), k=2, forced_topk=forced)
    assert out["counts"].tolist() == [0, 0, 0, 0, 0, 0, 4, 4]
    assert out["offsets"].tolist() == [0, 0, 0, 0, 0, 0, 0, 4, 8]
    sel = np.take_along_axis(out["probs"], forced.astype(np.int64), 1)
    assert np.allclose(out["topk_w"], sel / sel.sum(1, keepdims=True))


def test_rms_glue():
    h = np.float64([[3.0, -4.0, 0.0, 0.0]])
    assert np.allclose(O.rms_glue(h), [[3 / 2.5, -4 / 2.5, 0, 0]], rtol=1e-15)
    g = np.random.default_rng(6).normal(size=(5, 64))
    assert np.allclose(np.mean(O.rms_glue(g) ** 2, axis=1), 1.0, rtol=1e-14)


@pytest.mark.parametrize("mistake", ["drop_up", "sigmoid_sign", "down_transposed", "no_renorm"])
def test_pins_catch_planted_mistakes(mistake, monkeypatch):
    """Plant one plausible mistake in the checker (on the CPU) and see a pin fail."""
    if mistake == "drop_up":
        orig = O.expert_ffn_dense

        def bad(x, wg, wu, wd, offsets, perm, k):       # h = silu(g) only, the "* u" term lost
            return orig(x, wg, np.ones_like(O.widen(wu)) / np.sum(np.abs(O.widen(x))), wd, offsets, perm, k)
        monkeypatch.setattr(O, "expert_ffn_dense", bad)
        failing = test_layer_hand_worked_top1
    elif mistake == "sigmoid_sign":
        monkeypatch.setattr(O, "silu", lambda z: z / (1.0 + np.exp(z)))
        failing = test_layer_hand_worked_top1
    elif mistake == "down_transposed":
        orig = O.expert_ffn_dense

        def bad(x, wg, wu, wd, offsets, perm, k):
            return orig(x, wg, wu, np.swapaxes(O.widen(wd), 1, 2), offsets, perm, k)
        monkeypatch.setattr(O, "expert_ffn_dense", bad)
        failing = test_layer_hand_worked_top1
    else:
        orig = O.gate_weights
        monkeypatch.setattr(O, "gate_weights", lambda Wt, S, renorm=True: orig(Wt, S, False))
        failing = test_gate_weights_identities
    with pytest.raises(AssertionError):
        failing()
