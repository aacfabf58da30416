"""Helpers for the GPU parity tests: build a layer from seeded synthetic tensors, run the CPU
checker on host copies of the very same bits, compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import moe_oracle as O
from synth import workloads as W

Y_TOL = 2e-2        # max |y_gpu - y_oracle| <= Y_TOL * RMS(y_oracle)   (bf16 weights, fp32 accumulation)
W_TOL = 1e-5        # gate weights, fp32 vs fp64
TIE_GAP = 1e-4      # k-th vs (k+1)-th logit closer than this: the selection is not decided


def build(shape: W.LayerShape, T: int, *, layer=0, path=0, renorm=True, max_tokens=None, tensors=None):
    import paper_2503_00245_b200 as P
    dev = torch.device("cuda:0")
    t = tensors if tensors is not None else W.make_layer(shape, T, device=dev, layer=layer)
    host = {k: W.to_host_bits(v) for k, v in t.items()}
    kw = dict(d_model=shape.d_model, d_ff=shape.d_ff, n_experts=shape.n_experts, top_k=shape.top_k)
    lay = P.MoELayer.from_math_layout(kw, t, x_dtype=t["x"].dtype, renorm=renorm, path=path,
                                      max_tokens=max_tokens or max(T, 1))
    return lay, t, host


def experts_of(host):
    return {k: v for k, v in host.items() if k not in ("x", "w_router", "b_router")}


def oracle_layer(host, k, renorm=True, forced=None):
    return O.layer_forward(host["x"], host["w_router"], host["b_router"], experts_of(host), k, renorm, forced)


def to64(t: torch.Tensor) -> np.ndarray:
    return O.widen(W.to_host_bits(t))


def rms(a: np.ndarray) -> float:
    return float(np.sqrt(np.mean(np.square(a))))


def assert_close_rms(got: np.ndarray, want: np.ndarray, tol=Y_TOL, what="y"):
    scale = rms(want)
    err = float(np.max(np.abs(got - want))) if want.size else 0.0
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    assert err <= tol * scale, f"{what}: max abs err {err:.3e} > {tol} * rms {scale:.3e}"
    return err / scale if scale else 0.0


def assert_close_in_output_type(got: np.ndarray, want: np.ndarray, rms_tol=1e-2, mant_bits=8, what="y"):
    """Element by element: |got - want| <= half a unit in the last place of the output type at that value
    (bf16: 8 significant bits) + rms_tol * RMS(want).  The first term is what ANY implementation that rounds
    its result to the output type may lose; the second bounds everything upstream of that rounding.  At a
    few million outputs the largest |y| reaches 5.5-6.5 RMS, where half an ulp alone is 1.7e-2 to 2.5e-2 RMS."""
    scale = rms(want)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    mag = np.maximum(np.abs(want), np.abs(got))
    expo = np.floor(np.log2(np.maximum(mag, 1e-300)))
    half_ulp = np.exp2(expo - mant_bits)
    excess = np.abs(got - want) - half_ulp
    worst = float(np.max(excess)) / scale
    assert worst <= rms_tol, f"{what}: error exceeds the output type's rounding by {worst:.3e} * rms (> {rms_tol})"
    return worst


def assert_valid_tied_selection(sel, logits, k: int, t=0):
    """At a token whose k-th and (k+1)-th logits are closer than TIE_GAP the selection is not unique, but
    it is not free either (Eq. 3): the k experts are distinct, every expert whose logit lies more than
    TIE_GAP above the k-th largest must be in the set, and none whose logit lies more than TIE_GAP
    below it may be."""
    sel = [int(e) for e in sel]
    assert len(set(sel)) == k and all(0 <= e < len(logits) for e in sel), (t, sel)
    kth = float(np.sort(logits)[::-1][k - 1])
    for e, v in enumerate(logits):
        if v > kth + TIE_GAP:
            assert e in sel, f"token {t}: expert {e} (logit {v:.6f}, k-th {kth:.6f}) missing from {sel}"
    for e in sel:
        assert logits[e] >= kth - TIE_GAP, f"token {t}: expert {e} (logit {logits[e]:.6f}) is below the k-th {kth:.6f}"


def check_routing(idx_gpu: np.ndarray, w_gpu: np.ndarray, ora: dict, k: int):
    """Indices bit-exact except at near-ties; gate weights matched by expert id.  Returns the
    near-tie mask (tokens whose selection the arithmetic's precision decides)."""
    tie = O.near_tie_tokens(ora["logits"], k, TIE_GAP)
    S, w = ora["topk_idx"], ora["topk_w"]
    for t in range(S.shape[0]):
        if tie[t]:
            assert_valid_tied_selection(idx_gpu[t], ora["logits"][t], k, t)
            continue
        srt = -np.sort(-ora["logits"][t])
        if k > 1 and np.min(srt[:k - 1] - srt[1:k]) < TIE_GAP:      # order inside the set undecided
            assert set(idx_gpu[t].tolist()) == set(S[t].tolist()), (t, idx_gpu[t], S[t])
            order = [list(S[t]).index(e) for e in idx_gpu[t]]
            assert np.allclose(w_gpu[t], w[t][order], atol=W_TOL, rtol=0)
        else:
            assert idx_gpu[t].tolist() == S[t].tolist(), (t, idx_gpu[t], S[t])
            assert np.allclose(w_gpu[t], w[t], atol=W_TOL, rtol=0), (t, w_gpu[t], w[t])
    return tie


def check_layer(lay, t, host, k, renorm=True, tol=Y_TOL):
    """Run moe_layer_forward and compare routing and y with the checker (forced routing at near-ties)."""
    T = t["x"].shape[0]
    idx = torch.empty((T, k), dtype=torch.int32, device="cuda")
    w = torch.empty((T, k), dtype=torch.float32, device="cuda")
    y = lay.forward(t["x"], topk_idx=idx, topk_w=w)
    torch.cuda.synchronize()
    assert lay.check() == 0
    ora = oracle_layer(host, k, renorm)
    idx_h, w_h = idx.cpu().numpy(), w.cpu().numpy()
    tie = check_routing(idx_h, w_h, ora, k)
    if tie.any() or not np.array_equal(idx_h, ora["topk_idx"]):
        ora = oracle_layer(host, k, renorm, forced=idx_h)     # same sets (checked above), GPU's order
    rel = assert_close_rms(to64(y), ora["y"], tol)
    return rel, ora, y
