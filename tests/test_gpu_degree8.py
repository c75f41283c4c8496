"""GPU parity of degree p = 8 (one more level of Algorithm 1's recursion) against the CPU oracle,
through the C ABI."""
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check

pytestmark = pytest.mark.gpu


def _packed_gaussians(H, h, r, seed, dtype):
    """[Ga; Gb; Gc] for G1 and for G2: two tensors [H, 2h + r, r]."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    G1 = torch.randn(H, 2 * h + r, r, generator=g).to(dtype).cuda()
    G2 = torch.randn(H, 2 * h + r, r, generator=g).to(dtype).cuda()
    return G1, G2


def _oracle_gaussians(G1, G2, hi, h):
    a, b = G1[hi].double().cpu().numpy(), G2[hi].double().cpu().numpy()
    return [a[:h], b[:h], a[h:2 * h], b[h:2 * h], a[2 * h:], b[2 * h:]]


@pytest.mark.parametrize("r,b,n,dtype,path", [
    (16, 128, 384, "f32", psk.PATH_AUTO), (32, 256, 512, "f32", psk.PATH_AUTO), (64, 128, 256, "f32", psk.PATH_AUTO),
    (32, 128, 128, "f32", psk.PATH_AUTO), (32, 256, 768, "bf16", psk.PATH_CUDA_CORES), (64, 256, 512, "bf16", psk.PATH_AUTO),
    # bf16 storage, r <= 32: half sketches and the attention on them by tensor-core kernels
    (32, 256, 768, "bf16", psk.PATH_TENSOR_CORES), (16, 128, 640, "bf16", psk.PATH_AUTO), (32, 512, 1024, "bf16", psk.PATH_AUTO),
])
def test_forward_and_backward(r, b, n, dtype, path):
    # rows scaled down: (q.k)^8 with |q|^2 = h would leave fp32's comfortable range
    w = wl.small_workload(B=1, H=2, n=n, r=r, b=b, dtype=dtype, seed=500 + r)
    inp = wl.make_inputs(w, "cuda")
    tdt = inp["Q"].dtype
    Q, K = (inp["Q"].float() * 0.25).to(tdt), (inp["K"].float() * 0.25).to(tdt)
    V, dO = inp["V"], inp["dO"]
    G1, G2 = _packed_gaussians(w.H, 64, r, 600 + r, tdt)
    psk.profile_enable(True)
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, p=8, path=path)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, p=8, path=path)
    torch.cuda.synchronize()
    kernels = {name for name, _ in psk.profile_records()}
    psk.profile_enable(False)
    on_tc = dtype == "bf16" and r <= 32 and path != psk.PATH_CUDA_CORES
    assert ("tc_fwd_out_kernel" in kernels) == on_tc and (("fwd_out_kernel" in kernels) != on_tc)
    # on that route the deeper sketch runs on the tensor cores too, forward and backward
    assert ({"sk8_tc_fwd_kernel", "sk8_tc_bwd_kernel"} <= kernels) == on_tc and ("sketch8_kernel" in kernels) != on_tc
    for hi in range(w.H):
        q, k, v, g = (x[0, hi].double().cpu().numpy() for x in (Q, K, V, dO))
        Gs = _oracle_gaussians(G1, G2, hi, 64)
        Mq, Mk = orc.half_sketch_degree4(q, Gs), orc.half_sketch_degree4(k, Gs)
        O_ref, d_ref = orc.causal_attention_blocked_from_half_sketches(Mq, Mk, v, b)
        check("O", O[0, hi], O_ref, TOL[dtype])
        check("denom", den[0, hi], d_ref, TOL[dtype])
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), orc.causal_polysketch8_attention_backward(q, k, v, Gs, g)):
            check(name, got[0, hi], ref, TOL[dtype])


def test_sketch_call_and_refusals():
    w = wl.small_workload(B=1, H=1, n=128, r=16, b=128, dtype="f32", seed=501)
    inp = wl.make_inputs(w, "cuda")
    G1, G2 = _packed_gaussians(1, 64, 16, 601, torch.float32)
    X = inp["Q"] * 0.25
    shp = psk.binding.make_shape(X, G1, 16, 128, 8)
    M = torch.empty(1, 1, 128, 16, device="cuda")
    st = psk.lib().psk_sketch(psk.binding.byref(shp), psk.binding._ptr(X), psk.binding._ptr(G1), psk.binding._ptr(G2),
                              psk.binding._ptr(M), None, None)
    assert st == 0
    torch.cuda.synchronize()
    Mref = orc.half_sketch_degree4(X[0, 0].double().cpu().numpy(), _oracle_gaussians(G1, G2, 0, 64))
    check("M", M[0, 0], Mref, 1e-5)
    with pytest.raises(psk.PskError) as e:
        psk.causal_attn_fwd(X, X, inp["V"], G1, G2, 128, p=8, flags=psk.FLAG_LOCAL_EXACT)
    assert e.value.code == -2
    with pytest.raises(psk.PskError) as e:      # fp32 storage has no tensor-core route
        psk.causal_attn_fwd(X, X, inp["V"], G1, G2, 128, p=8, path=psk.PATH_TENSOR_CORES)
    assert e.value.code == -2


def test_kept_states_on_the_tensor_cores():
    r, b, n = 32, 256, 1024
    w = wl.small_workload(B=2, H=2, n=n, r=r, b=b, dtype="bf16", seed=510)
    inp = wl.make_inputs(w, "cuda")
    Q, K = (inp["Q"].float() * 0.25).bfloat16(), (inp["K"].float() * 0.25).bfloat16()
    V, dO = inp["V"], inp["dO"]
    G1, G2 = _packed_gaussians(w.H, 64, r, 611, torch.bfloat16)
    shp = psk.binding.make_shape(Q, G1, r, b, 8, flags=psk.FLAG_KEEP_STATES)
    ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True)), dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, p=8, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, p=8, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    assert psk.check(ws) == 0
    for bi, hi in ((0, 1), (1, 0)):
        q, k, v, g = (x[bi, hi].double().cpu().numpy() for x in (Q, K, V, dO))
        Gs = _oracle_gaussians(G1, G2, hi, 64)
        Mq, Mk = orc.half_sketch_degree4(q, Gs), orc.half_sketch_degree4(k, Gs)
        O_ref, d_ref = orc.causal_attention_blocked_from_half_sketches(Mq, Mk, v, b)
        check("O", O[bi, hi], O_ref, TOL["bf16"])
        check("denom", den[bi, hi], d_ref, TOL["bf16"])
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), orc.causal_polysketch8_attention_backward(q, k, v, Gs, g)):
            check(name, got[bi, hi], ref, TOL["bf16"])


def test_strided_views_and_one_shared_sketch_on_the_tensor_cores():
    # [B, n, H, h] storage viewed as [B, H, n, h]; one packed Gaussian set for all heads
    B, H, n, r, b = 2, 3, 512, 32, 256
    w = wl.small_workload(B=B, H=H, n=n, r=r, b=b, dtype="bf16", seed=520)
    inp = wl.make_inputs(w, "cuda")
    view = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    Q, K = (view((inp[k].float() * 0.25).bfloat16()) for k in ("Q", "K"))
    V, dO = view(inp["V"]), view(inp["dO"])
    assert not Q.is_contiguous()
    G1, G2 = _packed_gaussians(1, 64, r, 621, torch.bfloat16)
    psk.profile_enable(True)
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, p=8)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, p=8)
    torch.cuda.synchronize()
    kernels = {name for name, _ in psk.profile_records()}
    psk.profile_enable(False)
    assert {"sk8_tc_fwd_kernel", "sk8_tc_bwd_kernel", "tc_bwd_k_kernel"} <= kernels
    assert O.stride() == Q.stride() and dQ.stride() == Q.stride()
    Gs = _oracle_gaussians(G1, G2, 0, 64)
    for bi, hi in ((0, 0), (1, 2)):
        q, k, v, g = (x[bi, hi].double().cpu().numpy() for x in (Q, K, V, dO))
        Mq, Mk = orc.half_sketch_degree4(q, Gs), orc.half_sketch_degree4(k, Gs)
        O_ref, d_ref = orc.causal_attention_blocked_from_half_sketches(Mq, Mk, v, b)
        check("O", O[bi, hi], O_ref, TOL["bf16"])
        check("denom", den[bi, hi], d_ref, TOL["bf16"])
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), orc.causal_polysketch8_attention_backward(q, k, v, Gs, g)):
            check(name, got[bi, hi], ref, TOL["bf16"])
