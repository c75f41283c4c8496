"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by
element, on the same seeded inputs."""
import numpy as np
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check, g_slice, oracle_backward, oracle_forward, oracle_rows

pytestmark = pytest.mark.gpu


def _paths(dtype):
    return [psk.PATH_CUDA_CORES] if dtype == "f32" else [psk.PATH_CUDA_CORES, psk.PATH_AUTO]


@pytest.mark.parametrize("r", [16, 32, 64])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sketch_matches_oracle(r, dtype):
    w = wl.small_workload(H=2, n=256, r=r, dtype=dtype, seed=11 + r)
    inp = wl.make_inputs(w, "cuda")
    M, Phi = psk.sketch(inp["Q"], inp["G1"], inp["G2"], want_phi=True)
    for hi in range(w.H):
        X = wl.head_slice_f64(inp["Q"], 0, hi)
        Mref = orc.half_sketch(X, g_slice(inp["G1"], hi), g_slice(inp["G2"], hi))
        check("M", M[0, hi], Mref, 1e-5)
        check("Phi", Phi[0, hi], orc.self_tensor(Mref), 1e-5)


@pytest.mark.parametrize("r,b,n,dtype", [
    (16, 128, 384, "f32"), (32, 256, 768, "f32"), (64, 128, 256, "f32"), (32, 128, 128, "f32"),
    (32, 256, 1024, "bf16"), (64, 512, 1024, "bf16"), (16, 128, 640, "bf16"),
    (32, 128, 128, "bf16"), (32, 256, 256, "bf16"), (64, 512, 512, "bf16"),      # a single block: no prefix state at all
])
def test_forward_and_backward_small(r, b, n, dtype):
    w = wl.small_workload(B=2, H=2, n=n, r=r, b=b, dtype=dtype, seed=3 * r + b)
    inp = wl.make_inputs(w, "cuda")
    for path in _paths(dtype):
        O, den = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], b, path=path)
        dQ, dK, dV = psk.causal_attn_bwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], O, den,
                                         inp["dO"], b, path=path)
        torch.cuda.synchronize()
        for bi in range(w.B):
            for hi in range(w.H):
                O_ref, d_ref = oracle_forward(inp, bi, hi, b)
                check("O", O[bi, hi], O_ref, TOL[dtype])
                check("denom", den[bi, hi], d_ref, TOL[dtype])
                # the backward is checked at the library's own O/denom inputs' precision:
                # the oracle recomputes its forward in fp64 from the same stored Q, K, V
                g = oracle_backward(inp, bi, hi, b)
                for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), g):
                    check(name, got[bi, hi], ref, TOL[dtype])


@pytest.mark.parametrize("r,b,n,corr", [(32, 256, 1024, False), (16, 128, 512, True), (64, 512, 1024, True),
                                        (32, 256, 256, True)])
def test_backward_reading_the_forwards_states(r, b, n, corr):
    # PSK_FLAG_KEEP_STATES: forward and backward share one workspace; the backward skips the
    # prefix-state pass.  Values with a common mean direction exercise the centring.
    w = wl.small_workload(B=1, H=2, n=n, r=r, b=b, dtype="bf16", seed=61 + r, correlated=corr)
    inp = wl.make_inputs(w, "cuda")
    args = (inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"])
    shp = psk.binding.make_shape(inp["Q"], inp["G1"], r, b, flags=psk.FLAG_KEEP_STATES)
    ws = torch.empty(psk.workspace_bytes(shp, True), dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(*args, b, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    dQ, dK, dV = psk.causal_attn_bwd(*args, O, den, inp["dO"], b, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    assert psk.check(ws) == 0
    for hi in range(w.H):
        O_ref, d_ref = oracle_forward(inp, 0, hi, b)
        check("O", O[0, hi], O_ref, TOL["bf16"])
        check("denom", den[0, hi], d_ref, TOL["bf16"])
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), oracle_backward(inp, 0, hi, b)):
            check(name, got[0, hi], ref, TOL["bf16"])


def test_config0_full():
    w = wl.WORKLOADS["c0"]
    inp = wl.make_inputs(w, "cuda")
    O, den = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], w.b)
    O_ref, d_ref = oracle_forward(inp, 0, 0, w.b)
    check("O", O[0, 0], O_ref, TOL["f32"])
    check("denom", den[0, 0], d_ref, TOL["f32"])
    # and against the quadratic definition, not only the block algorithm
    Q, K, V = (wl.head_slice_f64(inp[k], 0, 0) for k in "QKV")
    O_def, _ = orc.causal_polysketch_attention(Q, K, V, g_slice(inp["G1"], 0), g_slice(inp["G2"], 0))
    check("O vs definition", O[0, 0], O_def, TOL["f32"])


def test_shared_sketch_and_strided_views():
    # one (G1, G2) pair for all heads (the paper shares the sketch within a layer), and
    # tensors that are views with non-trivial strides
    w = wl.small_workload(B=1, H=3, n=256, r=16, b=128, dtype="f32", seed=21)
    inp = wl.make_inputs(w, "cuda")
    G1, G2 = inp["G1"][:1].contiguous(), inp["G2"][:1].contiguous()
    big = {k: torch.zeros(1, 3, 256, 128, device="cuda")[..., :64] for k in ("Q", "K", "V", "dO")}
    for k in big:
        big[k].copy_(inp[k])
    O, den = psk.causal_attn_fwd(big["Q"], big["K"], big["V"], G1, G2, 128)
    dQ, dK, dV = psk.causal_attn_bwd(big["Q"], big["K"], big["V"], G1, G2, O, den, big["dO"], 128)
    shared = dict(inp, G1=G1, G2=G2)
    for hi in range(3):
        O_ref, _ = oracle_forward(shared, 0, hi, 128)
        check("O", O[0, hi], O_ref, 1e-4)
        for name, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), oracle_backward(shared, 0, hi, 128)):
            check(name, got[0, hi], ref, 1e-4)


def test_properties_on_device():
    w = wl.small_workload(B=1, H=2, n=512, r=32, b=256, dtype="f32", seed=31)
    inp = wl.make_inputs(w, "cuda")
    args = (inp["G1"], inp["G2"])
    O, den = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], *args, 256)
    assert (den >= 1).all()
    # block-size invariance (Section 3.1: b changes only the order of summation)
    O2, den2 = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], *args, 128)
    assert orc.rel_l2(O2.cpu().numpy(), O.cpu().numpy()) < 1e-5
    # causality: changing keys/values after position c leaves rows < c bit-identical
    c = 300
    K2, V2 = inp["K"].clone(), inp["V"].clone()
    K2[:, :, c:] = torch.randn_like(K2[:, :, c:])
    V2[:, :, c:] = 7.0
    O3, den3 = psk.causal_attn_fwd(inp["Q"], K2, V2, *args, 256)
    assert torch.equal(O3[:, :, :c], O[:, :, :c]) and torch.equal(den3[:, :, :c], den[:, :, :c])
    # V = 1: every output entry is (d - 1)/d
    ones = torch.ones_like(inp["V"])
    O4, den4 = psk.causal_attn_fwd(inp["Q"], inp["K"], ones, *args, 256)
    expect = ((den4.double() - 1) / den4.double())[..., None].expand_as(O4)
    assert orc.rel_l2(O4.double().cpu().numpy(), expect.cpu().numpy()) < 1e-5
    # run-twice determinism
    O5, _ = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], *args, 256)
    assert torch.equal(O5, O)


def test_device_status_word_is_clean():
    w = wl.small_workload(B=1, H=1, n=128, r=16, b=128, dtype="f32", seed=41)
    inp = wl.make_inputs(w, "cuda")
    shp = psk.binding.make_shape(inp["Q"], inp["G1"], 16, 128)
    ws = torch.empty(psk.workspace_bytes(shp, False), dtype=torch.uint8, device="cuda")
    psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 128, workspace=ws)
    assert psk.check(ws) == 0
    assert psk.last_launch_count() > 0


@pytest.mark.parametrize("r,b,n", [(32, 1024, 2048), (16, 384, 768), (64, 1024, 1024), (32, 640, 1280)])
@pytest.mark.parametrize("flags", [0, psk.FLAG_KEEP_STATES, psk.FLAG_LOCAL_EXACT | psk.FLAG_KEEP_STATES])
def test_many_tiles_per_block_on_the_tensor_cores(r, b, n, flags):
    # blocks of 3, 5 and 8 row tiles (the paper's own b = 1024 among them): the rings of state chunks,
    # the aliased tile buffers and the "last chunk" bookkeeping all depend on the tile count
    w = wl.small_workload(B=1, H=2, n=n, r=r, b=b, dtype="bf16", seed=7 * r + b)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, G1, G2, dO = (inp[k] for k in ("Q", "K", "V", "G1", "G2", "dO"))
    shp = psk.binding.make_shape(Q, G1, r, b, flags=flags)
    ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True)), dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, workspace=ws, flags=flags)
    grads = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, workspace=ws, flags=flags)
    assert psk.check(ws) == 0
    diag = "exact" if flags & psk.FLAG_LOCAL_EXACT else "LR"
    for hi in range(w.H):
        f = lambda k: wl.head_slice_f64(inp[k], 0, hi)
        g1, g2 = g_slice(G1, hi), g_slice(G2, hi)
        O_ref, d_ref = orc.causal_polysketch_attention_blocked(f("Q"), f("K"), f("V"), g1, g2, b, diagonal=diag)
        refs = (O_ref, d_ref) + tuple(orc.causal_polysketch_attention_backward_blocked(
            f("Q"), f("K"), f("V"), g1, g2, f("dO"), b, diagonal=diag))
        for nm, got, ref in zip(("O", "denom", "dQ", "dK", "dV"), (O, den) + tuple(grads), refs):
            check("%s[%d]" % (nm, hi), got[0, hi], ref, TOL["bf16"])


def test_strided_views_and_one_shared_sketch_on_the_tensor_cores():
    # [B, n, H, h] storage viewed as [B, H, n, h] (TMA maps with non-dense strides), one G pair for all heads
    B, H, n, r, b = 2, 3, 512, 32, 256
    w = wl.small_workload(B=B, H=H, n=n, r=r, b=b, dtype="bf16", seed=91)
    inp = wl.make_inputs(w, "cuda")
    view = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)      # same values, strides of [B, n, H, h]
    Q, K, V, dO = (view(inp[k]) for k in ("Q", "K", "V", "dO"))
    assert not Q.is_contiguous()
    G1, G2 = inp["G1"][:1].contiguous(), inp["G2"][:1].contiguous()
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b)
    dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b)
    assert O.stride() == Q.stride() and dQ.stride() == Q.stride()
    one = dict(inp, G1=G1, G2=G2)
    for bi, hi in ((0, 0), (1, 2)):
        O_ref, d_ref = oracle_forward(one, bi, hi, b)
        check("O", O[bi, hi], O_ref, TOL["bf16"])
        check("denom", den[bi, hi], d_ref, TOL["bf16"])
        for nm, got, ref in zip(("dQ", "dK", "dV"), (dQ, dK, dV), oracle_backward(one, bi, hi, b)):
            check(nm, got[bi, hi], ref, TOL["bf16"])


def test_binding_refuses_kept_states_without_a_workspace_and_strided_sketch_matrices():
    w = wl.small_workload(B=1, H=2, n=256, r=32, b=128, dtype="bf16", seed=92)
    inp = wl.make_inputs(w, "cuda")
    args = (inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 128)
    with pytest.raises(ValueError):
        psk.causal_attn_fwd(*args, flags=psk.FLAG_KEEP_STATES)
    Gs = torch.empty((2, 64, 64), dtype=torch.bfloat16, device="cuda")[:, :, :32]
    with pytest.raises(ValueError):
        psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], Gs, Gs, 128)
