"""A bounded device-side wait that runs out: the kernel returns, the status word reports it through
psk_check, later waits of the same thread block return at once, and the next regular call on the
same workspace is clean.  Nothing in this test hangs or traps the GPU: the wait is on a barrier
nobody completes, and it ends by its own clock after two milliseconds."""
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl

pytestmark = pytest.mark.gpu
ERR_TIMEOUT = -7


def test_wait_runs_out_and_is_reported():
    w = wl.small_workload(B=1, H=1, n=512, r=32, b=256, dtype="bf16", seed=11)
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, G1, G2 = (inp[k] for k in ("Q", "K", "V", "G1", "G2"))
    shp = psk.binding.make_shape(Q, G1, w.r, w.b)
    ws = torch.empty(psk.workspace_bytes(shp, False), dtype=torch.uint8, device="cuda")
    O1, den1 = psk.causal_attn_fwd(Q, K, V, G1, G2, w.b, workspace=ws)
    assert psk.check(ws) == 0
    limit = 2_000_000                                          # 2 ms
    first_ns, second_ns, failed1, failed2 = psk.binding.selftest_wait_timeout(ws, limit)
    assert failed1 == 128 and failed2 == 128                   # every thread gave up, twice
    assert limit <= first_ns < 50 * limit                      # by its clock, not by luck
    assert second_ns < limit // 4                              # the second wait did not wait again
    assert psk.check(ws) == ERR_TIMEOUT
    assert "gave up" in psk.binding.status_string(ERR_TIMEOUT)
    # the context is intact and the next call starts from a clean status word
    O2, den2 = psk.causal_attn_fwd(Q, K, V, G1, G2, w.b, workspace=ws)
    assert psk.check(ws) == 0
    assert torch.equal(O1, O2) and torch.equal(den1, den2)


def test_selftest_rejects_bad_arguments():
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(psk.binding.PskError):
        psk.binding.selftest_wait_timeout(ws, 10 ** 10)         # limit above 0.1 s
    with pytest.raises(psk.binding.PskError):
        psk.binding.selftest_wait_timeout(ws[:16], 1000)        # too small
