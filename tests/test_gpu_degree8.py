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


@pytest.mark.parametrize("r,b,n,dtype", [(16, 128, 384, "f32"), (32, 256, 512, "f32"), (64, 128, 256, "f32"),
                                         (32, 128, 128, "f32"), (32, 256, 768, "bf16")])
def test_forward_and_backward(r, b, n, dtype):
    # rows scaled down: (q.k)^8 with |q|^2 = h would leave fp32's comfortable range
    w = wl.small_workload(B=1, H=2, n=n, r=r, b=b, dtype=dtype, seed=500 + r)
    inp = wl.make_inputs(w, "cuda")
    tdt = inp["Q"].dtype
    Q, K = (inp["Q"].float() * 0.25).to(tdt), (inp["K"].float() * 0.25).to(tdt)
    V, dO = inp["V"], inp["dO"]
    G1, G2 = _packed_gaussians(w.H, 64, r, 600 + r, tdt)
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, p=8)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, p=8)
    torch.cuda.synchronize()
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
