"""psk_decode_step (the recurrent form: one token per call on a running state) against the
oracle's definition of causal Polysketch attention, row by row, and against the library's own
forward."""
import time

import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc
from parity_util import TOL, check, g_slice

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("r,dtype", [(16, "f32"), (32, "f32"), (64, "f32"), (32, "bf16")])
def test_steps_reproduce_the_rows_of_the_definition(r, dtype):
    n = 128
    w = wl.small_workload(B=2, H=2, n=n, r=r, b=128, dtype=dtype, seed=700 + r)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, G1, G2 = (inp[k] for k in ("Q", "K", "V", "G1", "G2"))
    state = psk.decode_state(w.B, w.H, r)
    O = torch.empty_like(Q)
    den = torch.empty(w.B, w.H, n, device="cuda")
    for t in range(n):
        o, d = psk.decode_step(Q[:, :, t].contiguous(), K[:, :, t].contiguous(), V[:, :, t].contiguous(), G1, G2, state)
        O[:, :, t] = o
        den[:, :, t] = d
    torch.cuda.synchronize()
    for bi in range(w.B):
        for hi in range(w.H):
            q, k, v = (wl.head_slice_f64(inp[x], bi, hi) for x in "QKV")
            O_ref, d_ref = orc.causal_polysketch_attention(q, k, v, g_slice(G1, hi), g_slice(G2, hi))
            check("O", O[bi, hi], O_ref, TOL[dtype])
            check("denom", den[bi, hi], d_ref, TOL[dtype])
    # the state after n tokens is the block algorithm's sum of per-block states (Section 3.1)
    q, k, v = (wl.head_slice_f64(inp[x], 0, 0) for x in "QKV")
    PhiK = orc.polysketch_non_negative(k, g_slice(G1, 0), g_slice(G2, 0))
    C = torch.cat([V[0, 0].double().cpu(), torch.ones(n, 1, dtype=torch.float64)], dim=1).numpy()
    check("state", state[0, 0], PhiK.T @ C, 1e-5 if dtype == "f32" else 1e-2)
    # and the library's own forward agrees with its recurrent form
    O_fwd, den_fwd = psk.causal_attn_fwd(Q, K, V, G1, G2, 128, path=psk.PATH_CUDA_CORES)
    assert orc.rel_l2(O.float().cpu().numpy(), O_fwd.float().cpu().numpy()) <= TOL[dtype]


def test_bad_arguments_and_step_time():
    w = wl.small_workload(B=32, H=12, n=128, r=32, b=128, dtype="bf16", seed=710)
    inp = wl.make_inputs(w, "cuda")
    q, k, v = (inp[x][:, :, 0].contiguous() for x in "QKV")
    state = psk.decode_state(32, 12, 32)
    with pytest.raises(ValueError):
        psk.decode_step(q, k, v, inp["G1"], inp["G2"], state[:, :6].contiguous())
    for _ in range(3):
        psk.decode_step(q, k, v, inp["G1"], inp["G2"], state)
    torch.cuda.synchronize()
    # device time of the kernel itself (events the library records around its launch): a Python
    # caller cannot issue steps as fast as they run
    psk.profile_enable(True)
    for _ in range(20):
        psk.decode_step(q, k, v, inp["G1"], inp["G2"], state)
    torch.cuda.synchronize()
    recs = [ms for name, ms in psk.profile_records() if name == "decode_step_kernel"]
    psk.profile_enable(False)
    assert len(recs) == 20
    us = 1e3 * sorted(recs)[len(recs) // 2]
    moved = 2 * state.numel() * 4                     # the state is read and written once
    print("decode step: %.1f us for 384 heads, %.0f GB/s of state traffic" % (us, moved / us / 1e3))
    assert torch.isfinite(state).all()
    assert moved / (us * 1e-6) > 2.0e12               # streams the state at more than 2 TB/s
