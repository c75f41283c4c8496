"""Run-to-run reproducibility of the tensor-core path on a workload of several thousand CTAs.

The kernels hand work between warps through mbarriers whose phases alternate; a handshake that
is only almost right (a barrier completing twice before its slowest waiter has looked, a buffer
refilled a moment early) shows up as a rare timeout or a rare wrong tile, and only when many CTAs
run at once.  Every kernel here is deterministic (fixed summation orders, no atomics), so repeated
calls on the same inputs must agree bit for bit, and the status word must stay clear."""
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("local", [False, True])
@pytest.mark.parametrize("r,b,n", [(32, 256, 16384), (16, 128, 4096), (64, 512, 8192)])
def test_repeated_calls_agree_bitwise(r, b, n, local):
    w = wl.small_workload(B=2, H=6, n=n, r=r, b=b, dtype="bf16", seed=700 + r)
    inp = wl.make_inputs(w, "cuda", with_dO=True)
    Q, K, V, G1, G2, dO = (inp[k] for k in ("Q", "K", "V", "G1", "G2", "dO"))
    flags = psk.FLAG_KEEP_STATES | (psk.FLAG_LOCAL_EXACT if local else 0)
    shp = psk.binding.make_shape(Q, G1, r, b, flags=flags)
    ws = torch.zeros(psk.workspace_bytes(shp, True), dtype=torch.uint8, device="cuda")
    first = None
    for it in range(8):
        O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, workspace=ws, flags=flags)
        dQ, dK, dV = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, workspace=ws, flags=flags)
        assert psk.check(ws) == 0, "a bounded device-side wait gave up in repetition %d" % it
        out = [t.clone() for t in (O, den, dQ, dK, dV)]
        if first is None:
            first = out
            for t in out:
                assert torch.isfinite(t).all()
        else:
            for name, a, c in zip(("O", "denom", "dQ", "dK", "dV"), first, out):
                assert torch.equal(a, c), "%s differs between repetition 0 and %d" % (name, it)


def test_recomputing_backward_agrees_with_kept_states():
    """Without the keep flag the backward rebuilds the prefix states and the forward rows itself;
    both routes are the same arithmetic up to the rounding of the stored O - c."""
    w = wl.small_workload(B=1, H=4, n=4096, r=32, b=256, dtype="bf16", seed=911)
    inp = wl.make_inputs(w, "cuda", with_dO=True)
    Q, K, V, G1, G2, dO = (inp[k] for k in ("Q", "K", "V", "G1", "G2", "dO"))
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, w.b)
    g_plain = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, w.b)
    shp = psk.binding.make_shape(Q, G1, w.r, w.b, flags=psk.FLAG_KEEP_STATES)
    ws = torch.zeros(psk.workspace_bytes(shp, True), dtype=torch.uint8, device="cuda")
    O2, den2 = psk.causal_attn_fwd(Q, K, V, G1, G2, w.b, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    g_kept = psk.causal_attn_bwd(Q, K, V, G1, G2, O2, den2, dO, w.b, workspace=ws, flags=psk.FLAG_KEEP_STATES)
    assert psk.check(ws) == 0
    for name, a, c in zip(("dQ", "dK", "dV"), g_plain, g_kept):
        rel = (a.double() - c.double()).norm() / c.double().norm()
        assert rel <= 1e-2, (name, float(rel))


def _time_step(B, n, reps=3):
    w = wl.small_workload(B=B, H=6, n=n, r=32, b=256, dtype="bf16", seed=17)
    inp = wl.make_inputs(w, "cuda", with_dO=True)
    Q, K, V, G1, G2, dO = (inp[k] for k in ("Q", "K", "V", "G1", "G2", "dO"))
    flags = psk.FLAG_KEEP_STATES
    shp = psk.binding.make_shape(Q, G1, 32, 256, flags=flags)
    ws = torch.empty(psk.workspace_bytes(shp, True), dtype=torch.uint8, device="cuda")
    best = float("inf")
    for _ in range(reps + 1):                      # first repetition: warm-up
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, 256, workspace=ws, flags=flags)
        psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, 256, workspace=ws, flags=flags)
        e1.record()
        torch.cuda.synchronize()
        if _ > 0:
            best = min(best, e0.elapsed_time(e1))
    assert psk.check(ws) == 0
    return best


def test_time_is_linear_in_the_context_length():
    """Section 3.1: the cost is linear in n at a fixed block size (exact attention would be
    quadratic): four times the context at the same batch and heads costs about four times as much."""
    t_1 = _time_step(B=25, n=16384)                # 150 heads: every SM has work in every kernel
    t_4 = _time_step(B=25, n=65536)
    assert 3.2 <= t_4 / t_1 <= 4.8, (t_1, t_4)
