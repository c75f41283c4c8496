"""Non-causal Polysketch attention (Section 3, first formula) on the tensor-core path against the
oracle's definition: forward and backward, with and without kept states, several cuts of the
sequence for the state sum, and independence of the launch granularity b."""
import numpy as np
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check, g_slice
from paper_2310_01655_b200.inputs import head_slice_f64

pytestmark = pytest.mark.gpu


def _run(inp, w, flags, segs=0, b=None):
    b = w.b if b is None else b
    Q, K, V, G1, G2, dO = (inp[k] for k in ("Q", "K", "V", "G1", "G2", "dO"))
    shp = psk.binding.make_shape(Q, G1, w.r, b, flags=flags, seq_segments=segs)
    ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True)), dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, workspace=ws, flags=flags, seq_segments=segs)
    assert psk.check(ws) == 0
    grads = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, workspace=ws, flags=flags, seq_segments=segs)
    assert psk.check(ws) == 0
    return (O, den) + tuple(grads)


@pytest.mark.parametrize("r,b,n", [(32, 256, 1024), (16, 128, 768), (64, 512, 1024), (32, 128, 2048)])
@pytest.mark.parametrize("keep", [False, True])
def test_matches_the_definition(r, b, n, keep):
    w = wl.small_workload(B=2, H=2, n=n, r=r, b=b, dtype="bf16", seed=50 + r)
    inp = wl.make_inputs(w, "cuda")
    flags = psk.FLAG_NONCAUSAL | (psk.FLAG_KEEP_STATES if keep else 0)
    got = _run(inp, w, flags)
    tol = TOL["bf16"]
    for bi, hi in ((0, 0), (1, 1)):
        f = lambda k: head_slice_f64(inp[k], bi, hi)
        G1, G2 = g_slice(inp["G1"], hi), g_slice(inp["G2"], hi)
        O_ref, d_ref = orc.polysketch_attention_linear(f("Q"), f("K"), f("V"), G1, G2)
        refs = (O_ref, d_ref) + tuple(orc.polysketch_attention_backward_linear(f("Q"), f("K"), f("V"), G1, G2, f("dO")))
        for nm, g, ref in zip(("O", "denom", "dQ", "dK", "dV"), got, refs):
            check("%s[%d,%d]" % (nm, bi, hi), g[bi, hi], ref, tol)
    assert (got[1] >= 1).all()


def test_first_row_sees_every_key_and_the_last_row_equals_the_causal_call():
    w = wl.small_workload(B=1, H=2, n=1024, r=32, b=256, dtype="bf16", seed=77)
    inp = wl.make_inputs(w, "cuda")
    O, den = _run(inp, w, psk.FLAG_NONCAUSAL)[:2]
    Oc, denc = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], w.b)
    assert (den[..., :-1] > denc[..., :-1]).all()
    assert torch.allclose(den[..., -1], denc[..., -1], rtol=2e-2)
    assert torch.allclose(O[..., -1, :].float(), Oc[..., -1, :].float(), rtol=5e-2, atol=5e-2)


@pytest.mark.parametrize("segs", [1, 2, 8])
def test_cuts_of_the_sequence_and_block_size_do_not_matter(segs):
    w = wl.small_workload(B=1, H=2, n=2048, r=32, b=256, dtype="bf16", seed=78)
    inp = wl.make_inputs(w, "cuda")
    base = _run(inp, w, psk.FLAG_NONCAUSAL, segs=1, b=256)
    other = _run(inp, w, psk.FLAG_NONCAUSAL, segs=segs, b=128)
    for nm, a, o in zip(("O", "denom", "dQ", "dK", "dV"), base, other):
        ref = a.double().cpu().numpy()
        err = orc.rel_l2(o.double().cpu().numpy(), ref)
        assert err <= TOL["bf16"] / 4, (nm, err)


def test_unsupported_combinations_are_refused():
    w = wl.small_workload(B=1, H=1, n=512, r=32, b=256, dtype="bf16", seed=3)
    inp = wl.make_inputs(w, "cuda")
    args = (inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 256)
    with pytest.raises(psk.binding.PskError):
        psk.causal_attn_fwd(*args, flags=psk.FLAG_NONCAUSAL | psk.FLAG_LOCAL_EXACT)
    with pytest.raises(psk.binding.PskError):
        psk.causal_attn_fwd(*args, flags=psk.FLAG_NONCAUSAL, path=psk.PATH_CUDA_CORES)
    wf = wl.small_workload(B=1, H=1, n=512, r=32, b=256, dtype="f32", seed=3)
    inf = wl.make_inputs(wf, "cuda")
    with pytest.raises(psk.binding.PskError):
        psk.causal_attn_fwd(inf["Q"], inf["K"], inf["V"], inf["G1"], inf["G2"], 256, flags=psk.FLAG_NONCAUSAL)
