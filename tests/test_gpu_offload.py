"""GPU tests of the host-resident-expert path (Eq. 8) and of the replacement metric (Eq. 4-5)."""
import os

import numpy as np
import pytest
import torch

from oracle import exrep_oracle as X
from oracle import moe_oracle as O
from oracle import offload_oracle as F
from synth import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


def make_stack(sh, n_layers, slots):
    import paper_2503_00245_b200 as P
    layers, host = [], []
    for l in range(n_layers):
        t = W.make_layer(sh, 1, device="cuda", layer=l)
        host.append({k: W.to_host_bits(v) for k, v in t.items() if k != "x"})
        layers.append({"w_router": t["w_router"], "b_router": t["b_router"],
                       "gud": P.pack_dense(t["w_gate"], t["w_up"], t["w_down"])})
    stack = P.OffloadedStack(sh.d_model, sh.d_ff, sh.n_experts, sh.top_k, slots, layers,
                             x_dtype=torch.bfloat16 if sh.x_dtype == "bf16" else torch.float32)
    return stack, host


@pytest.mark.parametrize("slots", [2, 4])
def test_stacked_decode_with_offload_matches_checker(slots):
    sh = W.LayerShape("t", 5, 256, 512, n_experts=8, top_k=2, x_dtype="bf16", bias="zipf")
    n_layers, steps = 3, 10
    stack, host = make_stack(sh, n_layers, slots)
    traces = [[] for _ in range(n_layers)]
    for step in range(steps):
        h0 = W.make_x(sh.with_(x_dtype="f32"), 1, device="cuda", step=step)[0].contiguous()
        h = h0.clone()
        sel = stack.step(h)
        torch.cuda.synchronize()
        assert stack.check() == 0
        # checker: same chain in fp64, layer by layer, fed the rounding points the kernels have
        hh = h0.cpu().numpy().astype(np.float64)
        for l in range(n_layers):
            u = O.rms_glue(hh[None])[0]
            u_b = torch.from_numpy(u.astype(np.float32)).to(torch.bfloat16)         # the layer input is bf16
            xin = W.to_host_bits(u_b[None])
            ex = {k: v for k, v in host[l].items() if k not in ("w_router", "b_router")}
            ora = O.layer_forward(xin, host[l]["w_router"], host[l]["b_router"], ex, sh.top_k)
            tie = O.near_tie_tokens(ora["logits"], sh.top_k, U.TIE_GAP)[0]
            if not tie:
                assert sel[l] == ora["topk_idx"][0].tolist(), (step, l, sel[l], ora["topk_idx"][0])
            else:
                U.assert_valid_tied_selection(sel[l], ora["logits"][0], sh.top_k, (step, l))
                ora = O.layer_forward(xin, host[l]["w_router"], host[l]["b_router"], ex, sh.top_k,
                                      forced_topk=np.int32([sel[l]]))
            hh = hh + ora["y"][0]                       # h += y in fp32 on the device, y not rounded in between
            traces[l].append(sel[l])
        got = h.cpu().numpy().astype(np.float64)
        # u is rounded to bf16 at the same place on both sides; what is left is fp32 vs fp64 arithmetic inside the
        # layers, amplified by at most n_layers
        U.assert_close_rms(got, hh, tol=U.Y_TOL, what=f"h after step {step}")
    # bookkeeping: fetches, bytes, hits and the final residents, exactly, on the GPU's own routing
    st = stack.stats()
    tot = {"n_fetch": 0, "bytes": 0, "hits": 0}
    for l in range(n_layers):
        sim = F.lru_cache_sim(traces[l], sh.n_experts, slots, stack.slot_bytes)
        for k in tot:
            tot[k] += sim[k]
        assert stack.resident(l) == sim["slots"][-1]
    assert (st["fetches"], st["bytes"], st["hits"]) == (tot["n_fetch"], tot["bytes"], tot["hits"])
    if slots == sh.top_k:          # capacity k: exactly the rule of Eq. 8
        for l in range(n_layers):
            eq8 = F.eq8_policy(traces[l])
            sim = F.lru_cache_sim(traces[l], sh.n_experts, slots, 1)
            assert [sorted(e for e, _ in f) for f in sim["fetches"]][1:] == eq8[1:]
    stack.close()


@pytest.mark.parametrize("p_stay", [0.12, 0.87])
def test_stacked_decode_with_prescribed_expert_sets(p_stay):
    """Replay of sticky routing traces under the rule of Eq. 8 (capacity = k): outputs against the checker told to
    use the same sets, traffic against the policy simulation, replacement ratio (Eq. 4-5) of the trace itself."""
    sh = W.LayerShape("t", 5, 256, 512, n_experts=8, top_k=2, x_dtype="bf16", bias="none")
    n_layers, steps, slots = 3, 12, 2
    stack, host = make_stack(sh, n_layers, slots)
    traces = [W.sticky_routing_trace(777 + l, steps, sh.n_experts, sh.top_k, p_stay).tolist() for l in range(n_layers)]
    for step in range(steps):
        h0 = W.make_x(sh.with_(x_dtype="f32"), 1, device="cuda", step=step)[0].contiguous()
        h = h0.clone()
        sel = [traces[l][step] for l in range(n_layers)]
        stack.step_trace(h, sel)
        torch.cuda.synchronize()
        assert stack.check() == 0
        hh = h0.cpu().numpy().astype(np.float64)
        for l in range(n_layers):
            u = O.rms_glue(hh[None])[0]
            u_b = torch.from_numpy(u.astype(np.float32)).to(torch.bfloat16)
            ex = {k: v for k, v in host[l].items() if k not in ("w_router", "b_router")}
            ora = O.layer_forward(W.to_host_bits(u_b[None]), host[l]["w_router"], host[l]["b_router"], ex, sh.top_k,
                                  forced_topk=np.int32([sel[l]]))
            hh = hh + ora["y"][0]
        U.assert_close_rms(h.cpu().numpy().astype(np.float64), hh, tol=U.Y_TOL, what=f"h after step {step}")
    st = stack.stats()
    tot = {"n_fetch": 0, "bytes": 0, "hits": 0}
    for l in range(n_layers):
        sim = F.lru_cache_sim(traces[l], sh.n_experts, slots, stack.slot_bytes)
        for k in tot:
            tot[k] += sim[k]
        assert stack.resident(l) == sim["slots"][-1]
        eq8 = F.eq8_policy(traces[l])
        assert [sorted(e for e, _ in f) for f in sim["fetches"]][1:] == eq8[1:]
    assert (st["fetches"], st["bytes"], st["hits"]) == (tot["n_fetch"], tot["bytes"], tot["hits"])
    # the device-side metric on the same traces
    tr = torch.tensor(traces, dtype=torch.int32, device="cuda")
    hsum = torch.zeros(1, dtype=torch.int64, device="cuda")
    from paper_2503_00245_b200 import binding as B
    B.moe_expert_replacements(tr, n_layers, steps, sh.top_k, sh.n_experts, hsum)
    torch.cuda.synchronize()
    want = sum(X.hard_replacements(X.activity_from_topk(np.int32(traces[l])[None], sh.n_experts))[1] for l in range(n_layers))
    assert int(hsum.item()) == want
    stack.close()


def test_offload_ensure_argument_errors():
    from paper_2503_00245_b200 import binding as B
    sh = W.LayerShape("t", 5, 256, 512, n_experts=8, top_k=2)
    stack, _ = make_stack(sh, 1, 3)
    for bad in ([0, 0], [0, 8], [-1, 2], [0, 1, 2, 3]):
        with pytest.raises(B.MoeError) as e:
            B.moe_offload_ensure(stack.off, 0, bad)
        assert e.value.status == 1
    with pytest.raises(B.MoeError):
        B.moe_offload_ensure(stack.off, 1, [0, 1])
    stack.close()


def test_expert_replacements_kernel_matches_eq4_and_fig5():
    from paper_2503_00245_b200 import binding as B
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    # the paper's worked example (Fig. 5): rebuild the selections from the activity matrices
    golden = os.path.join(os.path.dirname(__file__), "golden", "fig5_expert_activity.txt")
    blocks, cur = {}, None
    for line in open(golden):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            cur = blocks.setdefault(line[1:].split("]")[0], [])
        else:
            cur.append([int(v) for v in line.split()])
    for name, want in (("bles", 11), ("moe", 21)):
        A = np.array(blocks[name]).T                       # [T, E]
        S = np.stack([np.flatnonzero(r) for r in A]).astype(np.int32)[None]   # [1, T, 2]
        B.moe_expert_replacements(torch.from_numpy(S).cuda(), 1, S.shape[1], 2, 8, out)
        torch.cuda.synchronize()
        assert int(out.item()) // 2 == want
    # random traces against the checker
    for seed, (Bn, T, k, E) in enumerate([(3, 50, 2, 8), (1, 2, 1, 4), (4, 1000, 4, 16)]):
        S = np.stack([W.sticky_routing_trace(100 + seed * 10 + b, T, E, k, 0.6) for b in range(Bn)])
        B.moe_expert_replacements(torch.from_numpy(S).cuda(), Bn, T, k, E, out)
        torch.cuda.synchronize()
        _, H = X.hard_replacements(X.activity_from_topk(S, E))
        assert int(out.item()) == H


def test_delta_uniform_kernel_matches_checker():
    """Expert balance per layer (Section 3.3): integer counts exactly, the deviation from uniform against the
    checker's reading of it (the paper prints no formula: parity unpinned on both sides)."""
    from paper_2503_00245_b200 import binding as B
    for seed, (Bn, T, k, E) in enumerate([(3, 50, 2, 8), (1, 1, 1, 4), (24, 256, 2, 16)]):
        S = np.stack([W.sticky_routing_trace(300 + seed * 40 + b, T, E, k, 0.5) for b in range(Bn)]).astype(np.int32)
        counts = torch.zeros((Bn, E), dtype=torch.int64, device="cuda")
        delta = torch.zeros(Bn + 1, dtype=torch.float64, device="cuda")
        bad = torch.zeros(1, dtype=torch.int64, device="cuda")
        B.moe_delta_uniform(torch.from_numpy(S).cuda(), Bn, T, k, E, counts, delta, bad)
        torch.cuda.synchronize()
        A = X.activity_from_topk(S, E)
        assert counts.cpu().numpy().tolist() == A.sum(axis=1).tolist()
        want = [X.delta_uniform(A[b:b + 1]) for b in range(Bn)]
        got = delta.cpu().numpy()
        assert np.allclose(got[:Bn], want, rtol=0, atol=1e-12)
        assert abs(got[Bn] - float(np.mean(want))) <= 1e-12
        assert int(bad.item()) == 0
    # ids outside [0, E) are reported, not counted
    S = np.int32([[[0, 1], [9, 1], [-1, 0]]])
    counts = torch.zeros((1, 4), dtype=torch.int64, device="cuda")
    delta = torch.zeros(2, dtype=torch.float64, device="cuda")
    bad = torch.zeros(1, dtype=torch.int64, device="cuda")
    B.moe_delta_uniform(torch.from_numpy(S).cuda(), 1, 3, 2, 4, counts, delta, bad)
    torch.cuda.synchronize()
    assert counts.cpu().numpy().tolist() == [[2, 2, 0, 0]] and int(bad.item()) == 2


def test_expert_replacements_reads_rows_as_sets():
    """Eq. 4 is written on the 0/1 activity matrix: a repeated id in a row counts once, an id outside the
    range not at all."""
    from paper_2503_00245_b200 import binding as B
    S = np.int32([[[0, 0], [0, 1], [5, 1], [1, 1], [2, 3]]])      # E = 4: id 5 does not exist
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    B.moe_expert_replacements(torch.from_numpy(S).cuda(), 1, 5, 2, 4, out)
    torch.cuda.synchronize()
    A = np.zeros((1, 5, 4), dtype=np.int64)
    for t, row in enumerate(S[0]):
        for e in row:
            if 0 <= e < 4:
                A[0, t, e] = 1
    assert int(out.item()) == X.hard_replacements(A)[1]


def test_stacked_decode_with_offload_at_the_phone_shape():
    """The offload configuration at its real widths (d 2048, f 5632, E 16, 4 resident experts per layer), a few
    layers and steps: one expert is 69 MB, so a fetch is nine chunks, every chunk its own launch over a range of
    hidden units that waits for that chunk's copy, all launches of a layer adding into the same accumulators.
    Outputs against the fp64 chain, fetches / bytes / hits / residents against the cache simulation."""
    sh = W.PHONE_OFFLOAD
    n_layers, steps, slots = 4, 6, 4
    stack, host = make_stack(sh, n_layers, slots)
    torch.cuda.empty_cache()
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
            u_b = torch.from_numpy(u.astype(np.float32)).to(torch.bfloat16)
            xin = W.to_host_bits(u_b[None])
            ex = {k: v for k, v in host[l].items() if k not in ("w_router", "b_router")}
            R = O.router_logits(xin, host[l]["w_router"], host[l]["b_router"])
            tie = O.near_tie_tokens(R, sh.top_k, U.TIE_GAP)[0]
            if tie:
                U.assert_valid_tied_selection(sel[l], R[0], sh.top_k, (step, l))
            ora = O.layer_forward(xin, host[l]["w_router"], host[l]["b_router"], ex, sh.top_k,
                                  forced_topk=np.int32([sel[l]]) if tie else None)
            if not tie:
                assert sel[l] == ora["topk_idx"][0].tolist(), (step, l, sel[l], ora["topk_idx"][0])
            hh = hh + ora["y"][0]
            traces[l].append(sel[l])
        U.assert_close_rms(h.cpu().numpy().astype(np.float64), hh, tol=U.Y_TOL, what=f"h after step {step}")
    st = stack.stats()
    tot = {"n_fetch": 0, "bytes": 0, "hits": 0}
    for l in range(n_layers):
        sim = F.lru_cache_sim(traces[l], sh.n_experts, slots, stack.slot_bytes)
        for k in tot:
            tot[k] += sim[k]
        assert stack.resident(l) == sim["slots"][-1]
    assert (st["fetches"], st["bytes"], st["hits"]) == (tot["n_fetch"], tot["bytes"], tot["hits"])
    assert st["fetches"] > 0 and st["hits"] > 0          # both kinds of layer were met
    stack.close()
