"""CPU checker for the sparse MoE feed-forward layer.  TEST INFRASTRUCTURE ONLY.

This is a plain, slow, fp64 restatement of what the layer computes, written from
the paper so the GPU library can be compared against it.  Nothing in the product
path may import it: only the tests, the smoke check and the benchmark's timed CPU
baseline do.  It shares no code with the CUDA sources; it depends on numpy alone.

Conventions: T tokens, d = model width, f = expert hidden width, E experts, k
active experts per token, r = decomposition rank.  Row-vector maths, y = x @ W.
bf16 inputs arrive as uint16 bit patterns and are widened exactly to fp64; fp32
inputs are widened exactly too.  Every intermediate is fp64; nothing is blocked,
fused or reordered beyond what each cited passage states.

Pinned by tests (closed forms, invariants, brute force, library special cases):
router_logits, softmax, top_k, gate_weights, permute, expert_ffn_dense,
reconstruct, expert_ffn_wd, combine, layer_forward, rms_glue.
Parity unpinned: none of the above; the paper prints no numeric layer output, so
absolute values for a seed are pinned only through those properties.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------- inputs
def widen(a) -> np.ndarray:
    """Exact widening to fp64.  uint16 arrays are bf16 bit patterns (sign, 8 exponent
    bits, 7 mantissa bits = the upper half of an IEEE fp32)."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if a.dtype in (np.float32, np.float64):
        return a.astype(np.float64)
    raise TypeError(f"unsupported input dtype {a.dtype}")


# --------------------------------------------------------------------------- router
def router_logits(x, w_router, b_router=None) -> np.ndarray:
    """Router logits R[t, e] = sum_i x[t, i] * W_r[i, e] (+ b[e]): the (T, E) logits
    tensor the routing weights are computed from (Section 2.3, first paragraph)."""
    R = widen(x) @ widen(w_router)
    if b_router is not None:
        R = R + widen(b_router)[None, :]
    return R


def softmax(R: np.ndarray) -> np.ndarray:
    """Routing weights W = softmax(tau * R) over the expert axis (Eq. 2) with tau = 1
    at inference; the row maximum is subtracted first (no change to the value)."""
    z = R - R.max(axis=-1, keepdims=True)
    ez = np.exp(z)
    return ez / ez.sum(axis=-1, keepdims=True)


def top_k(W: np.ndarray, k: int) -> np.ndarray:
    """S = top_k(W, K) (Eq. 3): per token the k experts with the largest routing
    weight, listed by descending weight; equal weights go to the lower index."""
    T, E = W.shape
    S = np.zeros((T, k), dtype=np.int32)
    for t in range(T):
        order = sorted(range(E), key=lambda e: (-W[t, e], e))
        S[t] = order[:k]
    return S


def gate_weights(W: np.ndarray, S: np.ndarray, renorm: bool = True) -> np.ndarray:
    """Contribution of each selected expert (the gating mechanism, Section 1): its
    routing weight, rescaled so a token's k weights sum to one when renorm is set."""
    w = np.take_along_axis(W, S.astype(np.int64), axis=1)
    if renorm:
        w = w / w.sum(axis=1, keepdims=True)
    return w


def route(x, w_router, b_router, k: int, renorm: bool = True):
    """Eq. 2 then Eq. 3 then the gate weights.  Returns (R, W, S, w)."""
    R = router_logits(x, w_router, b_router)
    W = softmax(R)
    S = top_k(W, k)
    return R, W, S, gate_weights(W, S, renorm)


def near_tie_tokens(R: np.ndarray, k: int, gap: float = 1e-4) -> np.ndarray:
    """Tokens whose k-th and (k+1)-th largest logits differ by less than `gap`:
    there the selected set is not decided by the arithmetic's precision."""
    if k >= R.shape[1]:
        return np.zeros(R.shape[0], dtype=bool)
    srt = -np.sort(-R, axis=1)
    return (srt[:, k - 1] - srt[:, k]) < gap


# --------------------------------------------------------------------------- permutation
def permute(S: np.ndarray, n_experts: int):
    """Group the T*k (token, choice) pairs by expert: a stable counting sort.
    Pair p = t*k + j goes to a slot; slots of one expert are contiguous and ascend
    in p.  Returns counts[E], offsets[E+1] (exclusive scan), perm[slot] = p and
    inv[p] = slot.  (Token-choice routing hands each expert a discrete token subset,
    Section 2.1; the grouping itself is bookkeeping.)"""
    T, k = S.shape
    counts = np.zeros(n_experts, dtype=np.int32)
    for t in range(T):
        for j in range(k):
            counts[S[t, j]] += 1
    offsets = np.zeros(n_experts + 1, dtype=np.int32)
    for e in range(n_experts):
        offsets[e + 1] = offsets[e] + counts[e]
    cursor = offsets[:-1].copy()
    perm = np.zeros(T * k, dtype=np.int32)
    inv = np.zeros(T * k, dtype=np.int32)
    for t in range(T):
        for j in range(k):
            e = S[t, j]
            slot = cursor[e]
            cursor[e] += 1
            perm[slot] = t * k + j
            inv[t * k + j] = slot
    return counts, offsets, perm, inv


# --------------------------------------------------------------------------- experts
def silu(z: np.ndarray) -> np.ndarray:
    """z * sigmoid(z) = z / (1 + exp(-z))."""
    return z / (1.0 + np.exp(-z))


def expert_ffn_dense(x, w_gate, w_up, w_down, offsets, perm, top_k_: int) -> np.ndarray:
    """Per slot s (expert e, token t = perm[s] // k): the Llama-style gated FFN the
    experts use (Section 3.1), o_s = (silu(x_t W_g[e]) * (x_t W_u[e])) W_d[e].
    Only experts that received tokens are evaluated.  Returns o[T*k, d]."""
    X = widen(x)
    E = len(offsets) - 1
    out = np.zeros((len(perm), X.shape[1]), dtype=np.float64)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        tok = perm[lo:hi] // top_k_
        Xe = X[tok]
        g = Xe @ widen(w_gate[e])
        u = Xe @ widen(w_up[e])
        h = silu(g) * u
        out[lo:hi] = h @ widen(w_down[e])
    return out


def reconstruct(L, R) -> np.ndarray:
    """M = L x R (Eq. 1), formed in fp64 and not rounded."""
    return widen(L) @ widen(R)


def expert_ffn_wd(x, gL, gR, uL, uR, dL, dR, offsets, perm, top_k_: int) -> np.ndarray:
    """Weight-decomposed experts: every expert matrix is replaced by the product of
    its two factors (Eq. 1; all three matrices of each expert), then the dense FFN
    runs on the reconstructed matrices."""
    X = widen(x)
    E = len(offsets) - 1
    out = np.zeros((len(perm), X.shape[1]), dtype=np.float64)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        tok = perm[lo:hi] // top_k_
        Xe = X[tok]
        g = Xe @ reconstruct(gL[e], gR[e])
        u = Xe @ reconstruct(uL[e], uR[e])
        h = silu(g) * u
        out[lo:hi] = h @ reconstruct(dL[e], dR[e])
    return out


# --------------------------------------------------------------------------- combine
def combine(o: np.ndarray, w: np.ndarray, inv: np.ndarray) -> np.ndarray:
    """y[t] = sum_j w[t, j] * o[inv[t*k + j]], j ascending: each expert's output
    enters with the weight the gate gave it (Section 1, Section 2.1)."""
    T, k = w.shape
    y = np.zeros((T, o.shape[1]), dtype=np.float64)
    for t in range(T):
        for j in range(k):
            y[t] += w[t, j] * o[inv[t * k + j]]
    return y


# --------------------------------------------------------------------------- whole layer
def layer_forward(x, w_router, b_router, experts: dict, k: int, renorm: bool = True,
                  forced_topk=None) -> dict:
    """Router -> softmax -> top-k -> gate weights -> grouping -> selected experts'
    FFN -> gate-weighted sum.  `experts` holds w_gate/w_up/w_down, or the six WD
    factors.  With `forced_topk` the selection S is taken as given (used where the
    selection is a near-tie) and everything downstream follows from it."""
    R = router_logits(x, w_router, b_router)
    W = softmax(R)
    S = top_k(W, k) if forced_topk is None else np.asarray(forced_topk, dtype=np.int32)
    w = gate_weights(W, S, renorm)
    E = W.shape[1]
    counts, offsets, perm, inv = permute(S, E)
    if "w_gate" in experts:
        o = expert_ffn_dense(x, experts["w_gate"], experts["w_up"], experts["w_down"], offsets, perm, k)
    else:
        o = expert_ffn_wd(x, experts["gL"], experts["gR"], experts["uL"], experts["uR"],
                          experts["dL"], experts["dR"], offsets, perm, k)
    y = combine(o, w, inv)
    return {"logits": R, "probs": W, "topk_idx": S, "topk_w": w, "counts": counts,
            "offsets": offsets, "perm": perm, "inv": inv, "out_slots": o, "y": y}


# --------------------------------------------------------------------------- stack glue
def rms_glue(h: np.ndarray):
    """Glue between stacked layers (a pre-norm residual block without learned scale):
    u = h / sqrt(mean(h^2)) feeds the MoE layer, whose output is added back to h."""
    h = np.asarray(h, dtype=np.float64)
    return h / np.sqrt(np.mean(h * h, axis=-1, keepdims=True))
