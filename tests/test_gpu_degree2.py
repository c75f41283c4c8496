"""GPU parity of degree p = 2 (no sketch; exact (q.k)^2 attention by the block algorithm on
h^2 features) against the CPU oracle, through the C ABI."""
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("b,n,dtype,path", [
    (128, 384, "f32", psk.PATH_AUTO), (256, 512, "f32", psk.PATH_AUTO), (128, 128, "f32", psk.PATH_AUTO),
    (256, 768, "bf16", psk.PATH_CUDA_CORES),
    # bf16 storage: the tensor-core kernels with the rows as their own half sketch
    (256, 768, "bf16", psk.PATH_AUTO), (128, 128, "bf16", psk.PATH_TENSOR_CORES), (512, 2048, "bf16", psk.PATH_TENSOR_CORES),
])
def test_forward_and_backward(b, n, dtype, path):
    w = wl.small_workload(B=1, H=2, n=n, r=64, b=b, dtype=dtype, seed=300 + b)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    O, den = psk.causal_attn_fwd(Q, K, V, None, None, b, p=2, path=path)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, None, None, O, den, dO, b, p=2, path=path)
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


def test_kept_states_on_the_tensor_cores():
    b, n = 256, 1024
    w = wl.small_workload(B=2, H=2, n=n, r=64, b=b, dtype="bf16", seed=310)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, dO = (inp[k] for k in ("Q", "K", "V", "dO"))
    shp = psk.binding.make_shape(Q, None, 64, b, 2, flags=psk.FLAG_KEEP_STATES)
    ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True)), dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(Q, K, V, None, None, b, p=2, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, None, None, O, den, dO, b, p=2, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    assert psk.check(ws) == 0
    for bi, hi in ((0, 0), (1, 1)):
        q, k, v, g = (wl.head_slice_f64(inp[x], bi, hi) for x in ("Q", "K", "V", "dO"))
        O_ref, d_ref = orc.causal_degree2_attention_blocked(q, k, v, b)
        check("O", O[bi, hi], O_ref, TOL["bf16"])
        check("denom", den[bi, hi], d_ref, TOL["bf16"])
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), orc.causal_degree2_attention_backward(q, k, v, g)):
            check(name, got[bi, hi], ref, TOL["bf16"])


def test_degree2_needs_r_equal_h():
    w = wl.small_workload(B=1, H=1, n=128, r=32, b=128, dtype="bf16", seed=302)
    inp = wl.make_inputs(w, "cuda")
    with pytest.raises(psk.PskError) as e:      # r = 32 with p = 2
        psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 128, p=2)
    assert e.value.code == -2
    wf = wl.small_workload(B=1, H=1, n=128, r=64, b=128, dtype="f32", seed=303)
    inf = wl.make_inputs(wf, "cuda")
    with pytest.raises(psk.PskError) as e:      # fp32 storage has no tensor-core path
        psk.causal_attn_fwd(inf["Q"], inf["K"], inf["V"], None, None, 128, p=2, path=psk.PATH_TENSOR_CORES)
    assert e.value.code == -2
