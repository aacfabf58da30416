"""Conveniences over the C ABI: pack weights once, own a context and its workspace.

No arithmetic of the layer happens here; every call forwards to libcosmoe.so.
"""
from __future__ import annotations

import torch

from . import binding as B


def pack_dense(w_gate: torch.Tensor, w_up: torch.Tensor, w_down: torch.Tensor):
    """[E,d,f], [E,d,f], [E,f,d] bf16 (maths layout) -> gud [E,f,3,d]."""
    E, d, f = w_gate.shape
    gud = torch.empty((E, f, 3, d), dtype=torch.bfloat16, device=w_gate.device)
    B.moe_pack_dense(d, f, E, w_gate, w_up, w_down, gud)
    return gud


def pack_wd(gL, gR, uL, uR, dL, dR):
    """Eq. 1 factors in maths layout -> (wd_a [E,r,2,d], wd_b [E,f,2,r], wd_c [E,r,f], wd_d [E,d,r])."""
    E, d, r = gL.shape
    f = gR.shape[2]
    dev, bf = gL.device, torch.bfloat16
    wd_a = torch.empty((E, r, 2, d), dtype=bf, device=dev)
    wd_b = torch.empty((E, f, 2, r), dtype=bf, device=dev)
    wd_c = torch.empty((E, r, f), dtype=bf, device=dev)
    wd_d = torch.empty((E, d, r), dtype=bf, device=dev)
    B.moe_pack_wd(d, f, r, E, gL, gR, uL, uR, dL, dR, wd_a, wd_b, wd_c, wd_d)
    return wd_a, wd_b, wd_c, wd_d


class MoELayer:
    """One MoE layer's packed weights plus a context and workspace sized for up to max_tokens."""

    def __init__(self, d_model, d_ff, n_experts, top_k, w_router, b_router=None, *, dense=None, wd=None,
                 x_dtype=torch.bfloat16, renorm=True, path=B.MOE_PATH_AUTO, max_tokens=1, expert_slot=None):
        assert (dense is None) != (wd is None)
        self.d, self.f, self.E, self.k = d_model, d_ff, n_experts, top_k
        self.x_dtype = x_dtype
        self.device = w_router.device
        self.rank = 0 if wd is None else wd[0].shape[1]
        self.cfg = B.make_config(d_model, d_ff, n_experts, top_k, self.rank,
                                 B.MOE_F32 if x_dtype == torch.float32 else B.MOE_BF16, int(renorm), path)
        if dense is not None:
            self.weights = B.make_weights(w_router, b_router, gud=dense, expert_slot=expert_slot)
        else:
            self.weights = B.make_weights(w_router, b_router, wd_a=wd[0], wd_b=wd[1], wd_c=wd[2], wd_d=wd[3],
                                          expert_slot=expert_slot)
        self.ctx = B.moe_create(self.cfg)
        self.max_tokens = max_tokens
        self.ws = torch.empty(B.moe_workspace_bytes(self.cfg, max_tokens), dtype=torch.uint8, device=self.device)

    @classmethod
    def from_math_layout(cls, shape_kw: dict, tensors: dict, **kw):
        """tensors: the dict synth.workloads.make_layer returns (already on the device)."""
        if "w_gate" in tensors:
            dense, wd = pack_dense(tensors["w_gate"], tensors["w_up"], tensors["w_down"]), None
        else:
            dense, wd = None, pack_wd(*(tensors[n] for n in ("gL", "gR", "uL", "uR", "dL", "dR")))
        return cls(shape_kw["d_model"], shape_kw["d_ff"], shape_kw["n_experts"], shape_kw["top_k"],
                   tensors["w_router"], tensors["b_router"], dense=dense, wd=wd, **kw)

    def _need(self, T):
        if T > self.max_tokens:
            raise ValueError(f"T={T} exceeds max_tokens={self.max_tokens} this layer's workspace was sized for")

    # ---- step-by-step calls -------------------------------------------------------------
    def route(self, x, want_probs=False):
        T = x.shape[0]
        idx = torch.empty((T, self.k), dtype=torch.int32, device=self.device)
        w = torch.empty((T, self.k), dtype=torch.float32, device=self.device)
        probs = torch.empty((T, self.E), dtype=torch.float32, device=self.device) if want_probs else None
        B.moe_route(self.ctx, x, T, self.weights, idx, w, probs)
        return idx, w, probs

    def permute(self, topk_idx):
        T = topk_idx.shape[0]
        offsets = torch.empty(self.E + 1, dtype=torch.int32, device=self.device)
        perm = torch.empty(T * self.k, dtype=torch.int32, device=self.device)
        inv = torch.empty(T * self.k, dtype=torch.int32, device=self.device)
        B.moe_permute(self.ctx, topk_idx, T, offsets, perm, inv)
        return offsets, perm, inv

    def expert_ffn(self, x, offsets, perm):
        T = x.shape[0]
        self._need(T)
        out = torch.empty((T * self.k, self.d), dtype=torch.float32, device=self.device)
        B.moe_expert_ffn(self.ctx, x, T, self.weights, offsets, perm, out, self.ws)
        return out

    def combine(self, out_slots, topk_w, inv):
        T = topk_w.shape[0]
        y = torch.empty((T, self.d), dtype=self.x_dtype, device=self.device)
        B.moe_combine(self.ctx, out_slots, topk_w, inv, T, y)
        return y

    # ---- the whole layer ------------------------------------------------------------------
    def forward(self, x, y=None, topk_idx=None, topk_w=None):
        T = x.shape[0]
        self._need(T)
        if y is None:
            y = torch.empty((T, self.d), dtype=self.x_dtype, device=self.device)
        B.moe_layer_forward(self.ctx, x, T, self.weights, y, topk_idx, topk_w, self.ws)
        return y

    def check(self) -> int:
        return B.moe_check(self.ctx)

    def close(self):
        if self.ctx:
            B.moe_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class OffloadedStack:
    """n_layers stacked MoE layers whose experts live in pinned host memory (packed gud layout); the device
    keeps `slots` experts per layer.  Owns the pinned master copy, the device slots, a ctx and its workspace."""

    def __init__(self, d_model, d_ff, n_experts, top_k, slots, layers, x_dtype=torch.bfloat16, device="cuda", fp8=False):
        """layers: iterable of dicts with w_router, b_router and gud [E,f,3,d] (device tensors, consumed one by one).
        fp8: keep the host copies as FP8 codes + row scales (half the bytes per fetch)."""
        import ctypes
        self.fp8 = fp8
        self.d, self.f, self.E, self.k, self.slots = d_model, d_ff, n_experts, top_k, slots
        self.cfg = B.make_config(d_model, d_ff, n_experts, top_k, 0,
                                 B.MOE_F32 if x_dtype == torch.float32 else B.MOE_BF16, 1, B.MOE_PATH_STREAM)
        self.slot_bytes = d_ff * 3 * d_model * 2
        self.host, self.routers_t = [], []
        ptrs = []
        self.blob_bytes = d_ff * 3 * d_model + d_ff * 3 * 4 if fp8 else self.slot_bytes
        for lay in layers:
            if fp8:
                gud = lay["gud"]
                rows = n_experts * d_ff * 3
                codes = torch.empty((n_experts, d_ff * 3 * d_model), dtype=torch.uint8, device=gud.device)
                scales = torch.empty((n_experts, d_ff * 3), dtype=torch.float32, device=gud.device)
                B.moe_fp8_quantize_rows(gud, rows, d_model, codes, scales)
                hg = torch.empty((n_experts, self.blob_bytes), dtype=torch.uint8, pin_memory=True)
                hg[:, :d_ff * 3 * d_model].copy_(codes)
                hg[:, d_ff * 3 * d_model:].copy_(scales.view(torch.uint8).reshape(n_experts, -1))
                del codes, scales
            else:
                hg = torch.empty(lay["gud"].shape, dtype=torch.bfloat16, pin_memory=True)
                hg.copy_(lay["gud"])
            self.host.append(hg)
            self.routers_t.append((lay["w_router"], lay["b_router"]))
            ptrs += [hg.data_ptr() + e * self.blob_bytes for e in range(n_experts)]
        self.n_layers = len(self.host)
        torch.cuda.synchronize()
        self.device_slots = torch.empty(self.n_layers * slots * self.slot_bytes, dtype=torch.uint8, device=device)
        self.off = B.moe_offload_create(self.cfg, self.n_layers, slots, ptrs, self.device_slots, self.slot_bytes, fp8=fp8)
        self.ctx = B.moe_create(self.cfg)
        self.ws = torch.empty(B.moe_workspace_bytes(self.cfg, 1), dtype=torch.uint8, device=device)
        self.routers = (B.moe_weights * self.n_layers)()
        for l, (wr, br) in enumerate(self.routers_t):
            self.routers[l].w_router = wr.data_ptr()
            self.routers[l].b_router = br.data_ptr() if br is not None else None
        self._ctypes = ctypes

    def step(self, h):
        """h: fp32 [d] device tensor, updated in place.  Returns the per-layer selections."""
        return B.moe_stack_decode_step(self.off, self.ctx, self.routers, h, self.n_layers, self.k, self.ws)

    def step_trace(self, h, sel):
        """The same step with every layer's expert set given (sel [n_layers][k]); no host wait between layers."""
        B.moe_stack_decode_step_trace(self.off, self.ctx, self.routers, h, sel, self.ws)

    def stats(self):
        return B.moe_offload_stats(self.off)

    def resident(self, layer):
        return B.moe_offload_resident(self.off, layer, self.slots)

    def check(self):
        return B.moe_check(self.ctx)

    def close(self):
        if self.off:
            B.moe_offload_destroy(self.off)
            self.off = None
        if self.ctx:
            B.moe_destroy(self.ctx)
            self.ctx = None
