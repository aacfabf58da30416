"""ctypes binding of libcosmoe.so: same names as include/cosmoe.h, argument marshalling only.

Tensors are torch CUDA tensors (PyTorch owns device memory and streams); every step of the
layer runs in the library's kernels.  There is no CPU fallback: if the shared library is
missing or no B200 is present, calls fail.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcosmoe.so")

MOE_OK = 0
MOE_F32, MOE_BF16 = 0, 1
MOE_PATH_AUTO, MOE_PATH_STREAM, MOE_PATH_TENSOR = 0, 1, 2
MOE_STREAM_MAX_TOKENS = 16


class MoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib().moe_status_string(status).decode() if _LIB is not None else "?"
        extra = f" (cudaError {_lib().moe_last_cuda_error()})" if status == 4 else ""
        super().__init__(f"{where}: {msg}{extra}")


class moe_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("d_model", "d_ff", "n_experts", "top_k", "wd_rank", "x_dtype", "renorm", "path")]


class moe_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("w_router", "b_router", "gud", "wd_a", "wd_b", "wd_c", "wd_d", "expert_slot")]


_LIB = None
_P = C.c_void_p
_SIGS = {
    "moe_status_string": (C.c_char_p, [C.c_int]),
    "moe_last_cuda_error": (C.c_int, []),
    "moe_device_sm_count": (C.c_int, []),
    "moe_create": (C.c_int, [C.POINTER(moe_config), C.POINTER(_P)]),
    "moe_destroy": (C.c_int, [_P]),
    "moe_check": (C.c_int, [_P, _P]),
    "moe_workspace_bytes": (C.c_int, [C.POINTER(moe_config), C.c_int32, C.POINTER(C.c_size_t)]),
    "moe_launch_count": (C.c_int, [_P, C.POINTER(C.c_uint64)]),
    "moe_set_finaliser_wait": (C.c_int, [_P, C.c_longlong]),
    "moe_seed_arrival_counter": (C.c_int, [_P, C.c_ulonglong, _P]),
    "moe_pack_dense": (C.c_int, [C.c_int32] * 3 + [_P] * 5),
    "moe_pack_wd": (C.c_int, [C.c_int32] * 4 + [_P] * 11),
    "moe_route": (C.c_int, [_P, _P, C.c_int32, C.POINTER(moe_weights), _P, _P, _P, _P]),
    "moe_permute": (C.c_int, [_P, _P, C.c_int32, _P, _P, _P, _P]),
    "moe_expert_ffn": (C.c_int, [_P, _P, C.c_int32, C.POINTER(moe_weights), _P, _P, _P, _P, C.c_size_t, _P]),
    "moe_combine": (C.c_int, [_P, _P, _P, _P, C.c_int32, _P, _P]),
    "moe_layer_forward": (C.c_int, [_P, _P, C.c_int32, C.POINTER(moe_weights), _P, _P, _P, _P, C.c_size_t, _P]),
    "moe_layer_forward_static": (C.c_int, [C.POINTER(moe_config), _P, C.c_int32, C.POINTER(moe_weights), _P, _P, _P, _P]),
    "moe_offload_create": (C.c_int, [C.POINTER(moe_config), C.c_int32, C.c_int32, C.POINTER(_P), _P, C.c_size_t,
                                     C.POINTER(_P)]),
    "moe_offload_create_fp8": (C.c_int, [C.POINTER(moe_config), C.c_int32, C.c_int32, C.POINTER(_P), _P, C.c_size_t,
                                         C.POINTER(_P)]),
    "moe_fp8_quantize_rows": (C.c_int, [_P, C.c_int64, C.c_int32, _P, _P, _P]),
    "moe_fp8_dequantize_rows": (C.c_int, [_P, _P, C.c_int64, C.c_int32, _P, _P]),
    "moe_offload_destroy": (C.c_int, [_P]),
    "moe_offload_ensure": (C.c_int, [_P, C.c_int32, C.POINTER(C.c_int32), C.c_int32, _P]),
    "moe_offload_slot_table": (C.c_int, [_P, C.c_int32, C.POINTER(_P)]),
    "moe_offload_resident": (C.c_int, [_P, C.c_int32, C.POINTER(C.c_int32)]),
    "moe_offload_stats": (C.c_int, [_P, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]),
    "moe_stack_decode_step": (C.c_int, [_P, _P, C.POINTER(moe_weights), _P, C.POINTER(C.c_int32), _P, C.c_size_t, _P]),
    "moe_stack_decode_step_trace": (C.c_int, [_P, _P, C.POINTER(moe_weights), _P, C.POINTER(C.c_int32), _P, C.c_size_t,
                                              _P]),
    "moe_offload_host_times": (C.c_int, [_P, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_uint64)]),
    "moe_expert_replacements": (C.c_int, [_P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P, _P]),
    "moe_delta_uniform": (C.c_int, [_P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P, _P]),
}
EXPORTS = tuple(_SIGS)


def _lib():
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is not built: run `python -m paper_2503_00245_b200.build` "
                               "(there is no CPU fallback)")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _LIB = lib
    return _LIB


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    # device tensors, or pinned host tensors (mapped: the device reaches them at the same address)
    assert (t.is_cuda or t.is_pinned()) and t.is_contiguous(), "device-resident (or pinned host) contiguous tensors only"
    return t.data_ptr()


def _stream(stream=None) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ok(rc: int, where: str):
    if rc != MOE_OK:
        raise MoeError(rc, where)


def make_config(d_model, d_ff, n_experts, top_k, wd_rank=0, x_dtype=MOE_BF16, renorm=1, path=MOE_PATH_AUTO):
    return moe_config(d_model, d_ff, n_experts, top_k, wd_rank, x_dtype, renorm, path)


def make_weights(w_router=None, b_router=None, gud=None, wd_a=None, wd_b=None, wd_c=None, wd_d=None,
                 expert_slot=None) -> moe_weights:
    w = moe_weights(*[_ptr(t) for t in (w_router, b_router, gud, wd_a, wd_b, wd_c, wd_d, expert_slot)])
    w._keep = (w_router, b_router, gud, wd_a, wd_b, wd_c, wd_d, expert_slot)  # keep tensors alive
    return w


# ------------------------------------------------------------------ same names as the header
def moe_device_sm_count() -> int:
    return _lib().moe_device_sm_count()


def moe_create(cfg: moe_config) -> int:
    h = _P()
    _ok(_lib().moe_create(C.byref(cfg), C.byref(h)), "moe_create")
    return h.value


def moe_destroy(ctx: int):
    _ok(_lib().moe_destroy(ctx), "moe_destroy")


def moe_check(ctx: int, stream=None) -> int:
    return _lib().moe_check(ctx, _stream(stream))


def moe_workspace_bytes(cfg: moe_config, T: int) -> int:
    n = C.c_size_t()
    _ok(_lib().moe_workspace_bytes(C.byref(cfg), T, C.byref(n)), "moe_workspace_bytes")
    return n.value


def moe_set_finaliser_wait(ctx: int, cycles: int):
    _ok(_lib().moe_set_finaliser_wait(ctx, cycles), "moe_set_finaliser_wait")


def moe_seed_arrival_counter(ctx: int, value: int, stream=None):
    _ok(_lib().moe_seed_arrival_counter(ctx, value, _stream(stream)), "moe_seed_arrival_counter")


def moe_launch_count(ctx: int) -> int:
    n = C.c_uint64()
    _ok(_lib().moe_launch_count(ctx, C.byref(n)), "moe_launch_count")
    return n.value


def moe_pack_dense(d, f, n_experts, w_gate, w_up, w_down, gud_out, stream=None):
    _ok(_lib().moe_pack_dense(d, f, n_experts, _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(gud_out),
                              _stream(stream)), "moe_pack_dense")


def moe_pack_wd(d, f, r, n_experts, gL, gR, uL, uR, dL, dR, wd_a, wd_b, wd_c, wd_d, stream=None):
    _ok(_lib().moe_pack_wd(d, f, r, n_experts, *[_ptr(t) for t in (gL, gR, uL, uR, dL, dR, wd_a, wd_b, wd_c, wd_d)],
                           _stream(stream)), "moe_pack_wd")


def moe_route(ctx, x, T, w: moe_weights, topk_idx, topk_w, probs=None, stream=None):
    _ok(_lib().moe_route(ctx, _ptr(x), T, C.byref(w), _ptr(topk_idx), _ptr(topk_w), _ptr(probs), _stream(stream)),
        "moe_route")


def moe_permute(ctx, topk_idx, T, expert_offsets, perm, inv, stream=None):
    _ok(_lib().moe_permute(ctx, _ptr(topk_idx), T, _ptr(expert_offsets), _ptr(perm), _ptr(inv), _stream(stream)),
        "moe_permute")


def moe_expert_ffn(ctx, x, T, w: moe_weights, expert_offsets, perm, out_slots, ws, stream=None):
    _ok(_lib().moe_expert_ffn(ctx, _ptr(x), T, C.byref(w), _ptr(expert_offsets), _ptr(perm), _ptr(out_slots),
                              _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)), "moe_expert_ffn")


def moe_combine(ctx, out_slots, topk_w, inv, T, y, stream=None):
    _ok(_lib().moe_combine(ctx, _ptr(out_slots), _ptr(topk_w), _ptr(inv), T, _ptr(y), _stream(stream)),
        "moe_combine")


def moe_layer_forward(ctx, x, T, w: moe_weights, y, topk_idx=None, topk_w=None, ws=None, stream=None):
    _ok(_lib().moe_layer_forward(ctx, _ptr(x), T, C.byref(w), _ptr(y), _ptr(topk_idx), _ptr(topk_w), _ptr(ws),
                                 ws.numel() * ws.element_size(), _stream(stream)), "moe_layer_forward")


def moe_layer_forward_static(cfg: moe_config, x, T, w: moe_weights, y, topk_idx=None, topk_w=None, stream=None) -> int:
    """The layer without a ctx or workspace (nothing is allocated); returns the status instead of raising."""
    return _lib().moe_layer_forward_static(C.byref(cfg), _ptr(x), T, C.byref(w), _ptr(y), _ptr(topk_idx),
                                           _ptr(topk_w), _stream(stream))


def moe_offload_create(cfg: moe_config, n_layers, slots_per_layer, host_expert_ptrs, device_slots, slot_bytes,
                       fp8=False) -> int:
    """host_expert_ptrs: sequence of n_layers*E host addresses (pinned memory the caller keeps alive); with fp8 they
    point to FP8 blobs (codes, then row scales) and moe_offload_create_fp8 is called."""
    arr = (C.c_void_p * len(host_expert_ptrs))(*host_expert_ptrs)
    h = _P()
    fn = _lib().moe_offload_create_fp8 if fp8 else _lib().moe_offload_create
    _ok(fn(C.byref(cfg), n_layers, slots_per_layer, arr, _ptr(device_slots), slot_bytes, C.byref(h)),
        "moe_offload_create_fp8" if fp8 else "moe_offload_create")
    _KEEP[h.value] = arr
    return h.value


_KEEP = {}


def moe_offload_destroy(off: int):
    _KEEP.pop(off, None)
    _ok(_lib().moe_offload_destroy(off), "moe_offload_destroy")


def moe_offload_ensure(off: int, layer: int, topk_idx_host, stream=None):
    sel = (C.c_int32 * len(topk_idx_host))(*[int(v) for v in topk_idx_host])
    _ok(_lib().moe_offload_ensure(off, layer, sel, len(topk_idx_host), _stream(stream)), "moe_offload_ensure")


def moe_offload_slot_table(off: int, layer: int) -> int:
    p = _P()
    _ok(_lib().moe_offload_slot_table(off, layer, C.byref(p)), "moe_offload_slot_table")
    return p.value


def moe_offload_resident(off: int, layer: int, n_slots: int):
    out = (C.c_int32 * n_slots)()
    _ok(_lib().moe_offload_resident(off, layer, out), "moe_offload_resident")
    return list(out)


def moe_offload_stats(off: int):
    a, b, c = C.c_uint64(), C.c_uint64(), C.c_uint64()
    _ok(_lib().moe_offload_stats(off, C.byref(a), C.byref(b), C.byref(c)), "moe_offload_stats")
    return {"fetches": a.value, "bytes": b.value, "hits": c.value}


def moe_stack_decode_step(off: int, ctx: int, routers, h, n_layers: int, k: int, ws, stream=None):
    """routers: ctypes array of moe_weights (one per layer).  Returns the [n_layers][k] selection as a list."""
    trace = (C.c_int32 * (n_layers * k))()
    _ok(_lib().moe_stack_decode_step(off, ctx, routers, _ptr(h), trace, _ptr(ws), ws.numel() * ws.element_size(),
                                     _stream(stream)), "moe_stack_decode_step")
    return [list(trace[l * k:(l + 1) * k]) for l in range(n_layers)]


def moe_stack_decode_step_trace(off: int, ctx: int, routers, h, sel, ws, stream=None):
    """sel: [n_layers][k] nested list of the experts every layer has to use."""
    flat = [int(e) for row in sel for e in row]
    arr = (C.c_int32 * len(flat))(*flat)
    _ok(_lib().moe_stack_decode_step_trace(off, ctx, routers, _ptr(h), arr, _ptr(ws), ws.numel() * ws.element_size(),
                                           _stream(stream)), "moe_stack_decode_step_trace")


def moe_expert_replacements(topk_trace, B, T, k, n_experts, h_total_out, stream=None):
    _ok(_lib().moe_expert_replacements(_ptr(topk_trace), B, T, k, n_experts, _ptr(h_total_out), _stream(stream)),
        "moe_expert_replacements")


def moe_delta_uniform(topk_trace, B, T, k, n_experts, counts_out, delta_out, bad_out, stream=None):
    _ok(_lib().moe_delta_uniform(_ptr(topk_trace), B, T, k, n_experts, _ptr(counts_out), _ptr(delta_out),
                                 _ptr(bad_out), _stream(stream)), "moe_delta_uniform")


def moe_offload_host_times(off: int):
    a, b, n = C.c_double(), C.c_double(), C.c_uint64()
    _ok(_lib().moe_offload_host_times(off, C.byref(a), C.byref(b), C.byref(n)), "moe_offload_host_times")
    return {"poll_s": a.value, "issue_s": b.value, "polls": n.value}


def moe_fp8_quantize_rows(w, rows, n, codes, scales, stream=None):
    _ok(_lib().moe_fp8_quantize_rows(_ptr(w), rows, n, _ptr(codes), _ptr(scales), _stream(stream)), "moe_fp8_quantize_rows")


def moe_fp8_dequantize_rows(codes, scales, rows, n, w, stream=None):
    _ok(_lib().moe_fp8_dequantize_rows(_ptr(codes), _ptr(scales), rows, n, _ptr(w), _stream(stream)),
        "moe_fp8_dequantize_rows")
