"""Sequence-parallel prefix scan over block states (Section 3.1 notes that the prefix sums Z_l can be
computed in parallel): a head's blocks are cut into runs, a first pass leaves each run's total, a
second pass starts every run from the sum of the totals before it.  The result must not depend on the
number of runs beyond rounding; checked against the oracle and against the single-run result."""
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from parity_util import TOL, check, oracle_backward, oracle_forward

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("r,b,n,segs", [(32, 256, 2048, 2), (32, 256, 2048, 4), (32, 128, 1024, 8),
                                        (16, 128, 1024, 4), (64, 512, 2048, 2), (64, 512, 2048, 4)])
@pytest.mark.parametrize("keep", [False, True])
def test_runs_of_blocks_match_oracle_and_single_run(r, b, n, segs, keep):
    w = wl.small_workload(B=1, H=2, n=n, r=r, b=b, dtype="bf16", seed=31 + r + segs)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, G1, G2, dO = (inp[k] for k in ("Q", "K", "V", "G1", "G2", "dO"))
    flags = psk.FLAG_KEEP_STATES if keep else 0
    res = {}
    for s in (1, segs):
        shp = psk.binding.make_shape(Q, G1, r, b, flags=flags, seq_segments=s)
        ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, True)), dtype=torch.uint8,
                         device="cuda")
        O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, b, workspace=ws, flags=flags, seq_segments=s)
        assert psk.check(ws) == 0
        grads = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, dO, b, workspace=ws, flags=flags, seq_segments=s)
        assert psk.check(ws) == 0
        res[s] = (O, den) + tuple(grads)
    tol = TOL["bf16"]
    for hi in range(w.H):
        O_ref, d_ref = oracle_forward(inp, 0, hi, b)
        refs = (O_ref, d_ref) + tuple(oracle_backward(inp, 0, hi, b))
        for nm, got, one, ref in zip(("O", "denom", "dQ", "dK", "dV"), res[segs], res[1], refs):
            check("%s[%d] runs=%d" % (nm, hi, segs), got[0, hi], ref, tol)
            # the two summation orders differ by rounding only: far inside the tolerance
            check("%s[%d] runs=%d vs 1" % (nm, hi, segs), got[0, hi], one[0, hi].double().cpu().numpy(), tol / 4)


def test_segments_must_divide_the_blocks():
    w = wl.small_workload(B=1, H=1, n=768, r=32, b=256, dtype="bf16", seed=3)
    inp = wl.make_inputs(w, "cuda")
    with pytest.raises(psk.binding.PskError):
        psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 256, seq_segments=2)
