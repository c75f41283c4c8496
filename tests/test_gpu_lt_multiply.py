"""psk_lt_multiply (Section 3.1's block algorithm on arbitrary feature matrices) against the
oracle's block algorithm and against the dense triangle."""
import numpy as np
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from oracle import polysketch as orc

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("batch,n,m,k,b", [(2, 256, 48, 65, 64), (1, 384, 100, 17, 128), (3, 128, 7, 128, 32),
                                           (1, 96, 33, 1, 96), (1, 512, 256, 65, 256)])
def test_matches_oracle_and_dense_triangle(batch, n, m, k, b):
    g = torch.Generator(device="cpu").manual_seed(1000 + n + m)
    A, B = (torch.randn(batch, n, m, generator=g) for _ in range(2))
    C = torch.randn(batch, n, k, generator=g)
    out = psk.lt_multiply(A.cuda(), B.cuda(), C.cuda(), b).cpu().double().numpy()
    for i in range(batch):
        a, bb, c = (x[i].double().numpy() for x in (A, B, C))
        dense = np.tril(a @ bb.T) @ c
        assert orc.rel_l2(out[i], dense) < 1e-5
        assert orc.rel_l2(out[i], orc.lt_multiply_blocked(a, bb, c, b)) < 1e-5


def test_with_polysketch_features_it_is_the_attention_numerator():
    # A = phi'(Q), B = phi'(K) from psk_sketch, C = [V | 1]: numerators and normalisers of Section 3
    w = wl.small_workload(B=1, H=2, n=256, r=16, b=128, dtype="f32", seed=401)
    inp = wl.make_inputs(w, "cuda")
    _, PhiQ = psk.sketch(inp["Q"], inp["G1"], inp["G2"], want_phi=True)
    _, PhiK = psk.sketch(inp["K"], inp["G1"], inp["G2"], want_phi=True)
    C = torch.cat([inp["V"], torch.ones_like(inp["V"][..., :1])], dim=-1)
    N = psk.lt_multiply(PhiQ[0].contiguous(), PhiK[0].contiguous(), C[0].contiguous(), 128)
    O, den = psk.causal_attn_fwd(inp["Q"], inp["K"], inp["V"], inp["G1"], inp["G2"], 128)
    d = 1 + N[..., 64]
    assert orc.rel_l2(d.cpu().numpy(), den[0].cpu().numpy()) < 1e-5
    assert orc.rel_l2((N[..., :64] / d[..., None]).cpu().numpy(), O[0].cpu().numpy()) < 1e-5


def test_bad_arguments():
    A = torch.zeros(1, 64, 8, device="cuda")
    C = torch.zeros(1, 64, 4, device="cuda")
    with pytest.raises(psk.PskError) as e:
        psk.lt_multiply(A, A, C, 48)            # b not a multiple of 32
    assert e.value.code == -3
    with pytest.raises(psk.PskError) as e:
        psk.lt_multiply(A, A, torch.zeros(1, 64, 129, device="cuda"), 32)     # k > 128
    assert e.value.code == -3


# ---- the tensor-core instance (bf16 feature matrices) ----
@pytest.mark.parametrize("batch,n,m,b", [(2, 512, 128, 128), (1, 768, 192, 256), (2, 256, 64, 256), (1, 1024, 512, 256),
                                         (1, 128, 64, 128)])
def test_tensor_core_instance_matches_oracle(batch, n, m, b):
    g = torch.Generator(device="cpu").manual_seed(2000 + n + m)
    A, B = ((torch.randn(batch, n, m, generator=g) / m ** 0.5).bfloat16() for _ in range(2))
    C = torch.randn(batch, n, 64, generator=g).bfloat16()
    psk.profile_enable(True)
    out, ws = psk.lt_multiply_bf16(A.cuda(), B.cuda(), C.cuda(), b)
    torch.cuda.synchronize()
    kernels = {name for name, _ in psk.profile_records()}
    psk.profile_enable(False)
    assert psk.check(ws) == 0
    assert "lt_tc_rows_kernel" in kernels and ("lt_tc_state_kernel" in kernels) == (n > b)
    out = out.cpu().double().numpy()
    for i in range(batch):
        a, bb, c = (x[i].double().numpy() for x in (A, B, C))      # the bf16 values the kernels read
        ref = orc.lt_multiply_blocked(a, bb, c, b)
        # states and masked scores are rounded to bf16 once before they are multiplied: 2^-9 each
        assert orc.rel_l2(out[i], ref) < 1e-2
        assert orc.rel_l2(out[i], np.tril(a @ bb.T) @ c) < 1e-2
        # a row's first entries depend on few terms: check a tile's worth row by row as well
        for row in (0, 1, 127, min(128, n - 1), n - 1):
            assert np.allclose(out[i][row], ref[row], rtol=3e-2, atol=3e-2 * np.abs(ref[row]).max() + 1e-6)


def test_tensor_core_instance_bad_arguments():
    A = torch.zeros(1, 256, 64, device="cuda", dtype=torch.bfloat16)
    C = torch.zeros(1, 256, 64, device="cuda", dtype=torch.bfloat16)
    for args, code in (((A, A, C, 64), -3), ((A[:, :, :32].contiguous(), A[:, :, :32].contiguous(), C, 128), -3),
                       ((A, A, C[:, :, :32].contiguous(), 128), -3), ((A[:, :192].contiguous(), A[:, :192].contiguous(), C[:, :192].contiguous(), 128), -3)):
        with pytest.raises(psk.PskError) as e:
            psk.lt_multiply_bf16(*args)
        assert e.value.code == code
