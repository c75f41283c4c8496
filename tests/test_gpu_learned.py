"""Learnable sketch (Algorithm 2 of the appendix) on the GPU against the oracle: the half sketch, causal
attention on it forward and backward, with the gradients of every parameter group, also with exact
same-block weights (the paper's "learned + local" variant)."""
import numpy as np
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import binding, inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check
from paper_2310_01655_b200.inputs import head_slice_f64

pytestmark = pytest.mark.gpu


def make_net(g, h, r):
    m = 8 * r
    return {"g0": 1.0 + 0.1 * g.standard_normal(h), "c0": 0.1 * g.standard_normal(h),
            "W1": g.standard_normal((h, m)) / np.sqrt(h), "b1": 0.1 * g.standard_normal(m),
            "g1": 1.0 + 0.1 * g.standard_normal(m), "c1": 0.1 * g.standard_normal(m),
            "W2": g.standard_normal((m, r)) / np.sqrt(m), "b2": 0.1 * g.standard_normal(r),
            "W3": g.standard_normal((r, m)) / np.sqrt(r), "b3": 0.1 * g.standard_normal(m),
            "W4": 1.5 * g.standard_normal((m, r)) / np.sqrt(m), "b4": 0.1 * g.standard_normal(r)}


def nets(r, seed):
    g = np.random.default_rng(seed)
    P1, P2 = make_net(g, 64, r), make_net(g, 64, r)
    # the library reads fp32 parameters: the oracle gets exactly those values
    flat = binding.pack_learned_params(P1, P2)
    Q1, Q2 = binding.unpack_learned_params(flat.double().cpu(), 64, r)
    return flat, {k: v.numpy() for k, v in Q1.items()}, {k: v.numpy() for k, v in Q2.items()}


@pytest.mark.parametrize("r", [16, 32, 64])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_half_sketch(r, dtype):
    assert binding.learned_param_count(64, r) == 2 * 64 + 8 * 64 * r + 24 * r * r + 34 * r
    w = wl.small_workload(B=1, H=2, n=128, r=r, dtype=dtype, seed=60 + r)
    inp = wl.make_inputs(w, "cuda")
    flat, P1, P2 = nets(r, 1)
    M, Phi = binding.learned_sketch(inp["Q"], flat, r, want_phi=True)
    assert float(M.abs().max()) <= np.sqrt(r) * (1 + 1e-6)
    for hi in range(w.H):
        Mref = orc.learned_half_sketch(head_slice_f64(inp["Q"], 0, hi), P1, P2)
        check("M", M[0, hi], Mref, 2e-5)
        check("Phi", Phi[0, hi], orc.self_tensor(Mref), 4e-5)


@pytest.mark.parametrize("r,b,n", [(16, 128, 256), (32, 128, 384), (64, 256, 256)])
@pytest.mark.parametrize("dtype,path", [("f32", psk.PATH_AUTO), ("bf16", psk.PATH_CUDA_CORES), ("bf16", psk.PATH_AUTO)])
@pytest.mark.parametrize("local", [False, True])
def test_attention_forward_and_backward_with_parameter_gradients(r, b, n, dtype, path, local):
    # (bf16 storage, r <= 32: PATH_AUTO is the tensor-core route, networks and attention, with sketched
    # or exact same-block weights; everything else runs on the CUDA cores)
    w = wl.small_workload(B=2, H=2, n=n, r=r, b=b, dtype=dtype, seed=70 + r)
    inp = wl.make_inputs(w, "cuda")
    if local:
        # (q . k)^4 next to weights bounded by r^2: keep the exact pairs on the same scale
        inp["Q"], inp["K"] = (0.35 * inp["Q"].float()).to(inp["Q"].dtype), (0.35 * inp["K"].float()).to(inp["K"].dtype)
    flat, P1, P2 = nets(r, 2)
    flags = psk.FLAG_LOCAL_EXACT if local else 0
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    psk.profile_enable(True)
    O, den = binding.learned_attn_fwd(Q, K, V, flat, r, b, flags, path=path)
    dQ, dK, dV, dflat = binding.learned_attn_bwd(Q, K, V, flat, O, den, dO, r, b, flags, path=path)
    torch.cuda.synchronize()
    kernels = {name for name, _ in psk.profile_records()}
    psk.profile_enable(False)
    on_tc = dtype == "bf16" and r <= 32 and path != psk.PATH_CUDA_CORES
    assert ("tc_bwd_k_kernel" in kernels) == on_tc
    # on that route the networks run on the tensor cores too (dense layers and weight gradients)
    assert ({"ltc_dense_norm_kernel", "ltc_dense_bwd_norm_kernel", "ltc_wgrad_kernel"} <= kernels) == on_tc
    assert ("learned_sketch_bwd_kernel" in kernels) == (not on_tc)
    tol = TOL[dtype]
    diag = "exact" if local else "LR"
    g1_sum = {k: 0.0 for k in orc.NET_KEYS}
    g2_sum = {k: 0.0 for k in orc.NET_KEYS}
    for bi in range(w.B):
        for hi in range(w.H):
            f = lambda k: head_slice_f64(inp[k], bi, hi)
            O_ref, d_ref = orc.causal_learned_polysketch_attention_blocked(f("Q"), f("K"), f("V"), P1, P2, b, diagonal=diag)
            check("O", O[bi, hi], O_ref, tol)
            check("denom", den[bi, hi], d_ref, tol)
            gq, gk, gv, g1, g2 = orc.causal_learned_polysketch_attention_backward(f("Q"), f("K"), f("V"), P1, P2, f("dO"), b, diag)
            # the oracle's backward starts from its own fp64 forward, as the other parity tests do
            for nm, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), (gq, gk, gv)):
                check(nm, got[bi, hi], ref, tol)
            for k in orc.NET_KEYS:
                g1_sum[k] = g1_sum[k] + g1[k]
                g2_sum[k] = g2_sum[k] + g2[k]
    # parameter gradients are sums over the batch, the heads and both uses of the networks
    d1, d2 = binding.unpack_learned_params(dflat, 64, r)
    for which, (got, ref) in enumerate(((d1, g1_sum), (d2, g2_sum))):
        for k in orc.NET_KEYS:
            check("net %d %s" % (which + 1, k), got[k], ref[k], 5 * tol if dtype == "bf16" else 2e-3)


def _run_and_check(inp, w, flat, P1, P2, r, b, heads, tol, with_params, bwd_heads=None, passes=None):
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    psk.profile_enable(True)
    O, den = binding.learned_attn_fwd(Q, K, V, flat, r, b)
    dQ, dK, dV, dflat = binding.learned_attn_bwd(Q, K, V, flat, O, den, dO, r, b)
    torch.cuda.synchronize()
    records = [name for name, _ in psk.profile_records()]
    kernels = set(records)
    psk.profile_enable(False)
    assert {"ltc_dense_norm_kernel", "ltc_wgrad_kernel", "tc_bwd_k_kernel"} <= kernels
    if passes is not None:
        # one first-normalisation launch per pass and tensor (Q, K), three times: the forward call, the
        # backward call's half sketches (no kept states here) and its recomputation inside the chain rule
        assert records.count("ltc_ln0_kernel") == 6 * passes
    for t in (O, den, dQ, dK, dV, dflat):
        assert torch.isfinite(t.float()).all()
    g1_sum = {k: 0.0 for k in orc.NET_KEYS}
    g2_sum = {k: 0.0 for k in orc.NET_KEYS}
    for bi, hi in heads:
        f = lambda k: head_slice_f64(inp[k], bi, hi)
        O_ref, d_ref = orc.causal_learned_polysketch_attention_blocked(f("Q"), f("K"), f("V"), P1, P2, b, diagonal="LR")
        check("O[%d,%d]" % (bi, hi), O[bi, hi], O_ref, tol)
        check("denom[%d,%d]" % (bi, hi), den[bi, hi], d_ref, tol)
        if bwd_heads is not None and (bi, hi) not in bwd_heads:
            continue
        gq, gk, gv, g1, g2 = orc.causal_learned_polysketch_attention_backward(f("Q"), f("K"), f("V"), P1, P2, f("dO"), b, "LR")
        for nm, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), (gq, gk, gv)):
            check("%s[%d,%d]" % (nm, bi, hi), got[bi, hi], ref, tol)
        for k in orc.NET_KEYS:
            g1_sum[k] = g1_sum[k] + g1[k]
            g2_sum[k] = g2_sum[k] + g2[k]
    if with_params:
        d1, d2 = binding.unpack_learned_params(dflat, 64, r)
        for which, (got, ref) in enumerate(((d1, g1_sum), (d2, g2_sum))):
            for k in orc.NET_KEYS:
                check("net %d %s" % (which + 1, k), got[k], ref[k], 5 * tol)


def test_networks_in_several_passes_over_the_rows(monkeypatch):
    # the tensor-core networks walk the rows in chunks (2^20 by default); with 256-row chunks this small
    # input takes six passes per tensor, and the weight-gradient accumulators add up across them
    monkeypatch.setenv("PSK_LEARNED_CHUNK_ROWS", "256")
    r, b = 32, 128
    w = wl.small_workload(B=2, H=2, n=384, r=r, b=b, dtype="bf16", seed=91)
    inp = wl.make_inputs(w, "cuda")
    flat, P1, P2 = nets(r, 4)
    _run_and_check(inp, w, flat, P1, P2, r, b, [(bi, hi) for bi in range(2) for hi in range(2)], TOL["bf16"], True, passes=6)


@pytest.mark.parametrize("local", [False, True])
def test_strided_views_on_the_tensor_cores(local):
    # [B, n, H, h] storage viewed as [B, H, n, h]: the networks read and write rows by their strides,
    # the attention kernels through tensor maps with non-dense strides
    r, b = 32, 128
    w = wl.small_workload(B=2, H=3, n=384, r=r, b=b, dtype="bf16", seed=93)
    inp = wl.make_inputs(w, "cuda")
    view = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    scale = 0.35 if local else 1.0
    inp = dict(inp, Q=view((scale * inp["Q"].float()).bfloat16()), K=view((scale * inp["K"].float()).bfloat16()),
               V=view(inp["V"]), dO=view(inp["dO"]))
    assert not inp["Q"].is_contiguous()
    flat, P1, P2 = nets(r, 6)
    flags = psk.FLAG_LOCAL_EXACT if local else 0
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    O, den = binding.learned_attn_fwd(Q, K, V, flat, r, b, flags)
    dQ, dK, dV, dflat = binding.learned_attn_bwd(Q, K, V, flat, O, den, dO, r, b, flags)
    assert O.stride() == Q.stride() and dQ.stride() == Q.stride()
    diag = "exact" if local else "LR"
    for bi, hi in ((0, 0), (1, 2)):
        f = lambda k: head_slice_f64(inp[k], bi, hi)
        O_ref, d_ref = orc.causal_learned_polysketch_attention_blocked(f("Q"), f("K"), f("V"), P1, P2, b, diagonal=diag)
        check("O", O[bi, hi], O_ref, TOL["bf16"])
        check("denom", den[bi, hi], d_ref, TOL["bf16"])
        gq, gk, gv, _, _ = orc.causal_learned_polysketch_attention_backward(f("Q"), f("K"), f("V"), P1, P2, f("dO"), b, diag)
        for nm, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), (gq, gk, gv)):
            check(nm, got[bi, hi], ref, TOL["bf16"])


@pytest.mark.parametrize("local", [False, True])
def test_kept_states_on_the_tensor_cores(local):
    # one workspace for both calls: the backward reads the states the forward left there
    r, b = 32, 256
    w = wl.small_workload(B=2, H=2, n=1024, r=r, b=b, dtype="bf16", seed=94)
    inp = wl.make_inputs(w, "cuda")
    if local:
        inp["Q"], inp["K"] = (0.35 * inp["Q"].float()).bfloat16(), (0.35 * inp["K"].float()).bfloat16()
    flat, P1, P2 = nets(r, 7)
    flags = psk.FLAG_KEEP_STATES | (psk.FLAG_LOCAL_EXACT if local else 0)
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    ws = torch.empty(binding.learned_workspace_bytes(Q, r, b, flags), dtype=torch.uint8, device="cuda")
    psk.profile_enable(True)
    O, den = binding.learned_attn_fwd(Q, K, V, flat, r, b, flags, ws)
    dQ, dK, dV, dflat = binding.learned_attn_bwd(Q, K, V, flat, O, den, dO, r, b, flags, ws)
    torch.cuda.synchronize()
    records = [name for name, _ in psk.profile_records()]
    kernels = set(records)
    psk.profile_enable(False)
    assert psk.check(ws) == 0
    assert "tc_bwd_prep_kernel" in kernels and "tc_bwd_recompute_kernel" not in kernels      # the kept states were used
    # ... and the kept half sketches: they were formed once per tensor, by the forward call
    assert records.count("ltc_combine_kernel") == 2
    diag = "exact" if local else "LR"
    for bi, hi in ((0, 1), (1, 0)):
        f = lambda k: head_slice_f64(inp[k], bi, hi)
        O_ref, d_ref = orc.causal_learned_polysketch_attention_blocked(f("Q"), f("K"), f("V"), P1, P2, b, diagonal=diag)
        check("O", O[bi, hi], O_ref, TOL["bf16"])
        check("denom", den[bi, hi], d_ref, TOL["bf16"])
        gq, gk, gv, _, _ = orc.causal_learned_polysketch_attention_backward(f("Q"), f("K"), f("V"), P1, P2, f("dO"), b, diag)
        for nm, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), (gq, gk, gv)):
            check(nm, got[bi, hi], ref, TOL["bf16"])


def test_networks_across_the_default_chunk_boundary():
    # 4 x 12 heads of 32768 rows: 1.5 M rows per tensor, so the second pass starts at head (2, 8)
    r, b = 32, 256
    w = wl.small_workload(B=4, H=12, n=32768, r=r, b=b, dtype="bf16", seed=92)
    inp = wl.make_inputs(w, "cuda")
    flat, P1, P2 = nets(r, 5)
    _run_and_check(inp, w, flat, P1, P2, r, b, [(2, 7), (2, 8), (3, 11)], TOL["bf16"], False, bwd_heads=[(2, 8)], passes=2)


def test_refusals():
    w = wl.small_workload(B=1, H=1, n=256, r=32, b=128, dtype="f32", seed=5)
    inp = wl.make_inputs(w, "cuda")
    flat, _, _ = nets(32, 3)
    with pytest.raises(psk.PskError):
        binding.learned_attn_fwd(inp["Q"], inp["K"], inp["V"], flat, 32, 128, psk.FLAG_NONCAUSAL)
    with pytest.raises(psk.PskError):
        binding.learned_attn_fwd(inp["Q"], inp["K"], inp["V"], flat, 32, 100)
    with pytest.raises(psk.PskError):            # fp32 storage has no tensor-core route
        binding.learned_attn_fwd(inp["Q"], inp["K"], inp["V"], flat, 32, 128, path=psk.PATH_TENSOR_CORES)
    assert binding.learned_param_count(48, 32) == 0
