"""8-bit expert storage on the host link: the device's FP8 E4M3 codes and row scales bit for bit against the CPU
checker, the widening back to bf16 bit for bit, and the stacked decode with FP8 host copies against the fp64 chain
run on the checker's own de-quantised weights."""
import numpy as np
import pytest
import torch

from oracle import fp8_oracle as Q
from oracle import moe_oracle as O
from oracle import offload_oracle as F
from synth import rng
from synth import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,n,sigma", [(64, 256, 0.06), (3 * 40, 2048, 0.02), (7, 8, 1.0), (33, 1440, 5.0)])
def test_codes_scales_and_widening_are_bit_exact(rows, n, sigma):
    from paper_2503_00245_b200 import binding as B
    w = rng.normal(4711 + rows, (rows, n), sigma, torch.bfloat16, "cuda")
    w[0, :] = 0                                              # an all-zero row: scale 1, codes 0
    if rows > 2:
        w[1, :] = w[1, :] * 1e-3                             # a row whose small values land in the subnormal codes
        w[1, 0] = 1.0
    codes = torch.empty((rows, n), dtype=torch.uint8, device="cuda")
    scales = torch.empty(rows, dtype=torch.float32, device="cuda")
    B.moe_fp8_quantize_rows(w, rows, n, codes, scales)
    back = torch.empty_like(w)
    B.moe_fp8_dequantize_rows(codes, scales, rows, n, back)
    torch.cuda.synchronize()
    bits = W.to_host_bits(w)
    c_ref, s_ref = Q.quantize_rows(bits)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    got = codes.cpu().numpy()
    zero = ((got | c_ref) & 0x7F) == 0                       # -0 and +0 are the same value
    assert np.array_equal(got[~zero], c_ref[~zero])
    want_back = Q.dequantize_rows(got, s_ref)
    gb = W.to_host_bits(back)
    nz = (gb & 0x7FFF) != 0
    assert np.array_equal(gb[nz], want_back[nz]) and not (want_back[~nz] & 0x7FFF).any()


def _math_layout_from_gud(gud_bits, d, f, E):
    g = gud_bits.reshape(E, f, 3, d)
    return {"w_gate": np.ascontiguousarray(g[:, :, 0, :].transpose(0, 2, 1)),
            "w_up": np.ascontiguousarray(g[:, :, 1, :].transpose(0, 2, 1)),
            "w_down": np.ascontiguousarray(g[:, :, 2, :])}


@pytest.mark.parametrize("sh,n_layers,steps,slots", [
    (W.LayerShape("t", 5, 256, 512, n_experts=8, top_k=2, x_dtype="bf16", bias="zipf"), 3, 8, 3),
    (W.LayerShape("t", 5, 1024, 2816, n_experts=8, top_k=2, x_dtype="bf16", bias="zipf"), 2, 4, 2),   # several chunks per fetch
])
def test_stacked_decode_with_fp8_host_copies(sh, n_layers, steps, slots):
    import paper_2503_00245_b200 as P
    d, f, E, k = sh.d_model, sh.d_ff, sh.n_experts, sh.top_k
    layers, host = [], []
    for l in range(n_layers):
        t = W.make_layer(sh, 1, device="cuda", layer=l)
        gud = P.pack_dense(t["w_gate"], t["w_up"], t["w_down"])
        gb = W.to_host_bits(gud).reshape(E * f * 3, d)
        c, s = Q.quantize_rows(gb)                                       # the checker's own 8-bit copy ...
        ex = _math_layout_from_gud(Q.dequantize_rows(c, s), d, f, E)      # ... and what the layer must compute with
        ex.update({"w_router": W.to_host_bits(t["w_router"]), "b_router": W.to_host_bits(t["b_router"])})
        host.append(ex)
        layers.append({"w_router": t["w_router"], "b_router": t["b_router"], "gud": gud})
    stack = P.OffloadedStack(d, f, E, k, slots, layers, fp8=True)
    assert stack.blob_bytes == f * 3 * d + f * 12
    traces = [[] for _ in range(n_layers)]
    for step in range(steps):
        h0 = W.make_x(sh.with_(x_dtype="f32"), 1, device="cuda", step=step)[0].contiguous()
        h = h0.clone()
        sel = stack.step(h)
        torch.cuda.synchronize()
        assert stack.check() == 0
        hh = h0.cpu().numpy().astype(np.float64)
        for l in range(n_layers):
            u = O.rms_glue(hh[None])[0]
            xin = W.to_host_bits(torch.from_numpy(u.astype(np.float32)).to(torch.bfloat16)[None])
            ex = {kk: v for kk, v in host[l].items() if kk not in ("w_router", "b_router")}
            R = O.router_logits(xin, host[l]["w_router"], host[l]["b_router"])
            tie = O.near_tie_tokens(R, k, U.TIE_GAP)[0]
            if tie:
                U.assert_valid_tied_selection(sel[l], R[0], k, (step, l))
            ora = O.layer_forward(xin, host[l]["w_router"], host[l]["b_router"], ex, k,
                                  forced_topk=np.int32([sel[l]]) if tie else None)
            if not tie:
                assert sel[l] == ora["topk_idx"][0].tolist()
            hh = hh + ora["y"][0]
            traces[l].append(sel[l])
        U.assert_close_rms(h.cpu().numpy().astype(np.float64), hh, tol=U.Y_TOL, what=f"h after step {step}")
    st = stack.stats()
    tot = {"n_fetch": 0, "bytes": 0, "hits": 0}
    for l in range(n_layers):
        sim = F.lru_cache_sim(traces[l], E, slots, stack.blob_bytes)
        for kk in tot:
            tot[kk] += sim[kk]
        assert stack.resident(l) == sim["slots"][-1]
    assert (st["fetches"], st["bytes"], st["hits"]) == (tot["n_fetch"], tot["bytes"], tot["hits"])
    # the prescribed-set step over the same object
    h = W.make_x(sh.with_(x_dtype="f32"), 1, device="cuda", step=99)[0].contiguous()
    stack.step_trace(h, [[0, 1]] * n_layers)
    torch.cuda.synchronize()
    assert stack.check() == 0 and bool(torch.isfinite(h).all())
    stack.close()
