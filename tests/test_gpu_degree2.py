"""GPU parity of degree p = 2 (no sketch; exact (q.k)^2 attention by the block algorithm on
h^2 features) against the CPU oracle, through the C ABI."""
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("b,n,dtype", [(128, 384, "f32"), (256, 512, "f32"), (128, 128, "f32"), (256, 768, "bf16")])
def test_forward_and_backward(b, n, dtype):
    w = wl.small_workload(B=1, H=2, n=n, r=64, b=b, dtype=dtype, seed=300 + b)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    O, den = psk.causal_attn_fwd(Q, K, V, None, None, b, p=2)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, None, None, O, den, dO, b, p=2)
    torch.cuda.synchronize()
    for hi in range(w.H):
        q, k, v, g = (wl.head_slice_f64(inp[x], 0, hi) for x in ("Q", "K", "V", "dO"))
        O_ref, d_ref = orc.causal_degree2_attention_blocked(q, k, v, b)
        check("O", O[0, hi], O_ref, TOL[dtype])
        check("denom", den[0, hi], d_ref, TOL[dtype])
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), orc.causal_degree2_attention_backward(q, k, v, g)):
            check(name, got[0, hi], ref, TOL[dtype])


def test_sketch_call_returns_rows_and_their_tensor_square():
    w = wl.small_workload(B=1, H=1, n=128, r=64, b=128, dtype="f32", seed=301)
    inp = wl.make_inputs(w, "cuda")
    M, Phi = psk.sketch(inp["Q"], None, None, want_phi=True)
    x = wl.head_slice_f64(inp["Q"], 0, 0)
    check("M", M[0, 0], x, 1e-6)
    check("Phi", Phi[0, 0], orc.self_tensor(x), 1e-6)


def test_degree2_needs_r_equal_h_and_the_cuda_core_kernels():
    w = wl.small_workload(B=1, H=1, n=128, r=32, b=128, dtype="bf16", seed=302)
    inp = wl.make_inputs(w, "cuda")
    with pytest.raises(psk.PskError) as e:      # r = 32 with p = 2
        psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 128, p=2)
    assert e.value.code == -2
    with pytest.raises(psk.PskError) as e:
        psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], None, None, 128, p=2, path=psk.PATH_TENSOR_CORES)
    assert e.value.code == -2
