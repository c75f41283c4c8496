"""GPU parity of PSK_FLAG_LOCAL_EXACT (exact polynomial weights inside a block, Section 3.2)
against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check, g_slice

pytestmark = pytest.mark.gpu

LOCAL = psk.FLAG_LOCAL_EXACT


def _oracle(inp, bi, hi, b, backward):
    Q, K, V = (wl.head_slice_f64(inp[k], bi, hi) for k in "QKV")
    G1, G2 = g_slice(inp["G1"], hi), g_slice(inp["G2"], hi)
    fwd = orc.causal_polysketch_attention_blocked(Q, K, V, G1, G2, b, diagonal="exact")
    if not backward:
        return fwd, None
    dO = wl.head_slice_f64(inp["dO"], bi, hi)
    return fwd, orc.causal_polysketch_attention_backward_blocked(Q, K, V, G1, G2, dO, b, diagonal="exact")


@pytest.mark.parametrize("r,b,n,dtype", [
    (16, 128, 384, "f32"), (32, 256, 768, "f32"), (64, 128, 256, "f32"),
    (32, 128, 128, "f32"),                                     # a single block: exact degree-4 attention
    (32, 256, 1024, "bf16"), (64, 512, 1024, "bf16"), (16, 128, 640, "bf16"), (32, 256, 256, "bf16"),
])
def test_forward_and_backward_small(r, b, n, dtype):
    w = wl.small_workload(B=2, H=2, n=n, r=r, b=b, dtype=dtype, seed=5 * r + b)
    inp = wl.make_inputs(w, "cuda")
    args = (inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"])
    # bf16 storage: the tensor-core kernels (PATH_AUTO) and the CUDA-core kernels
    for path in ([psk.PATH_CUDA_CORES] if dtype == "f32" else [psk.PATH_CUDA_CORES, psk.PATH_AUTO]):
        O, den = psk.causal_attn_fwd(*args, b, path=path, flags=LOCAL)
        dQ, dK, dV = psk.causal_attn_bwd(*args, O, den, inp["dO"], b, path=path, flags=LOCAL)
        torch.cuda.synchronize()
        for bi in range(w.B):
            for hi in range(w.H):
                (O_ref, d_ref), g = _oracle(inp, bi, hi, b, True)
                check("O", O[bi, hi], O_ref, TOL[dtype])
                check("denom", den[bi, hi], d_ref, TOL[dtype])
                for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), g):
                    check(name, got[bi, hi], ref, TOL[dtype])


def test_single_block_is_exact_polynomial_attention():
    # b = n: no pair goes through the sketch; compare with Section 2.1's definition directly
    w = wl.small_workload(B=1, H=2, n=256, r=16, b=256, dtype="f32", seed=77)
    inp = wl.make_inputs(w, "cuda")
    O, den = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 256, flags=LOCAL)
    for hi in range(2):
        Q, K, V = (wl.head_slice_f64(inp[k], 0, hi) for k in "QKV")
        O_ref, d_ref = orc.causal_exact_polynomial_attention(Q, K, V, 4)
        check("O", O[0, hi], O_ref, 1e-4)
        check("denom", den[0, hi], d_ref, 1e-4)


def test_flag_changes_only_same_block_pairs():
    w = wl.small_workload(B=1, H=1, n=512, r=32, b=128, dtype="f32", seed=78)
    inp = wl.make_inputs(w, "cuda")
    args = (inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"])
    O_plain, _ = psk.causal_attn_fwd(*args, 128)
    O_loc, den = psk.causal_attn_fwd(*args, 128, flags=LOCAL)
    assert orc.rel_l2(O_loc.cpu().numpy(), O_plain.cpu().numpy()) > 1e-3      # the flag is not ignored
    assert (den >= 1).all()
    # the result now depends on the block size (through which pairs are exact)
    O_256, _ = psk.causal_attn_fwd(*args, 256, flags=LOCAL)
    assert orc.rel_l2(O_256.cpu().numpy(), O_loc.cpu().numpy()) > 1e-3
    # causality survives
    c = 300
    K2, V2 = inp["K"].clone(), inp["V"].clone()
    K2[:, :, c:] = torch.randn_like(K2[:, :, c:])
    V2[:, :, c:] = 7.0
    O3, den3 = psk.causal_attn_fwd(inp["Q"], K2, V2, inp["G1"], inp["G2"], 128, flags=LOCAL)
    assert torch.equal(O3[:, :, :c], O_loc[:, :, :c]) and torch.equal(den3[:, :, :c], den[:, :, :c])


@pytest.mark.parametrize("r,b,n,corr", [(32, 256, 1024, False), (16, 128, 512, True), (64, 512, 1024, True),
                                        (32, 256, 256, True), (32, 512, 2048, False)])
def test_tensor_core_backward_reading_the_forwards_states(r, b, n, corr):
    # both flags: forward and backward share one workspace on the tensor-core path
    w = wl.small_workload(B=1, H=2, n=n, r=r, b=b, dtype="bf16", seed=91 + r, correlated=corr)
    inp = wl.make_inputs(w, "cuda")
    args = (inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"])
    flags = psk.FLAG_KEEP_STATES | LOCAL
    shp = psk.binding.make_shape(inp["Q"], inp["G1"], r, b, path=psk.PATH_TENSOR_CORES, flags=flags)
    ws = torch.empty(psk.workspace_bytes(shp, True), dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(*args, b, path=psk.PATH_TENSOR_CORES, workspace=ws, flags=flags)
    dQ, dK, dV = psk.causal_attn_bwd(*args, O, den, inp["dO"], b, path=psk.PATH_TENSOR_CORES, workspace=ws, flags=flags)
    assert psk.check(ws) == 0
    for hi in range(w.H):
        (O_ref, d_ref), g = _oracle(inp, 0, hi, b, True)
        check("O", O[0, hi], O_ref, TOL["bf16"])
        check("denom", den[0, hi], d_ref, TOL["bf16"])
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), g):
            check(name, got[0, hi], ref, TOL["bf16"])


@pytest.mark.parametrize("name", ["c2", "c3"])
def test_full_size_configuration(name):
    """PSK_FLAG_LOCAL_EXACT at a benchmark configuration's full size, as `bench.py --local-exact`
    runs it: sampled (batch, head) slices against the block-form oracle, finiteness of the full
    tensors."""
    w = wl.WORKLOADS[name]
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, G1, G2 = (inp[k] for k in ("Q", "K", "V", "G1", "G2"))
    flags = psk.FLAG_KEEP_STATES | LOCAL
    shp = psk.binding.make_shape(Q, G1, w.r, w.b, flags=flags)
    ws = torch.empty(psk.workspace_bytes(shp, True), dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, w.b, workspace=ws, flags=flags)
    grads = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, inp["dO"], w.b, workspace=ws, flags=flags)
    assert psk.check(ws) == 0
    for t in (O, den) + tuple(grads):
        assert torch.isfinite(t).all()
    assert (den >= 1).all()
    for bi, hi in ((0, 0), (w.B - 1, w.H - 1)):
        (O_ref, d_ref), g = _oracle(inp, bi, hi, w.b, True)
        check("O[%d,%d]" % (bi, hi), O[bi, hi], O_ref, TOL["bf16"])
        check("denom[%d,%d]" % (bi, hi), den[bi, hi], d_ref, TOL["bf16"])
        for nm, got, ref in zip(("dQ", "dK", "dV"), grads, g):
            check("%s[%d,%d]" % (nm, bi, hi), got[bi, hi], ref, TOL["bf16"])
