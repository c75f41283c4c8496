"""The allocation-free forward (psk_causal_attn_fwd_static) against the regular forward.

Some users of the library run where device allocation is off limits: inside a host
application that owns all GPU memory through its own pool, or in a loop that may not
call the allocator.  For them the library carries its scratch as a fixed 16 MiB array.
This file is collected last so that a failure here cannot hide any other test."""
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import check, oracle_forward

pytestmark = pytest.mark.gpu


def _rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm())


@pytest.mark.parametrize("dtype,tol", [("f32", 1e-4), ("bf16", 2e-2)])
def test_static_scratch_forward_matches_regular_forward_twice(dtype, tol):
    assert psk.static_scratch_bytes() == 16 << 20
    # two calls in a row with different inputs and shapes: the array keeps the first call's
    # bytes, and the second result must not depend on them
    for seed, n, r, b in ((51, 512, 32, 256), (52, 384, 16, 128)):
        w = wl.small_workload(B=1, H=2, n=n, r=r, b=b, dtype=dtype, seed=seed)
        inp = wl.make_inputs(w, "cuda")
        args = (inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], b)
        O = torch.full_like(inp["Q"], float("nan"))
        den = torch.full((w.B, w.H, w.n), float("nan"), device="cuda")
        # first call: also lets the CUDA runtime load this shape's kernels (lazy module
        # loading takes device memory once and is not an allocation made by the call)
        psk.causal_attn_fwd_static(*args, out=O, denom=den)
        torch.cuda.synchronize()
        O.fill_(float("nan")); den.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        psk.causal_attn_fwd_static(*args, out=O, denom=den)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before        # the call allocated nothing
        O_ref, den_ref = psk.causal_attn_fwd(*args, path=psk.PATH_CUDA_CORES)
        torch.cuda.synchronize()
        assert torch.isfinite(O.float()).all() and torch.isfinite(den).all()
        assert _rel(O, O_ref) <= tol and _rel(den, den_ref) <= tol
        # and against the oracle itself, not only against the library's other entry point
        for hi in range(w.H):
            O_orc, d_orc = oracle_forward(inp, 0, hi, b)
            check("static O[%d]" % hi, O[0, hi], O_orc, tol)
            check("static denom[%d]" % hi, den[0, hi], d_orc, tol)


def test_static_scratch_degree_two_takes_no_sketch_matrices():
    # p = 2 reads no G1, G2: null pointers are valid here as they are for the regular forward
    w = wl.small_workload(B=1, H=2, n=256, r=64, b=128, dtype="f32", seed=54)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V = 0.5 * inp["Q"], 0.5 * inp["K"], inp["V"]
    O, den = psk.causal_attn_fwd_static(Q, K, V, None, None, 128, p=2)
    torch.cuda.synchronize()
    for hi in range(w.H):
        f = lambda t: t[0, hi].double().cpu().numpy()
        O_ref, d_ref = orc.causal_degree2_attention_blocked(f(Q), f(K), f(V), 128)
        check("static p=2 O[%d]" % hi, O[0, hi], O_ref, 1e-4)
        check("static p=2 denom[%d]" % hi, den[0, hi], d_ref, 1e-4)


def test_static_scratch_refuses_oversized_problems():
    w = wl.small_workload(B=2, H=4, n=4096, r=64, b=512, dtype="bf16", seed=53)
    inp = wl.make_inputs(w, "cuda", with_dO=False)
    with pytest.raises(psk.PskError) as e:
        psk.causal_attn_fwd_static(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 512)
    assert e.value.code == -5
