"""Parity of loma_rope_apply (through the C ABI) with the oracle's rotary embedding at the
layout's position ids.  fp32: max |delta| <= 1e-5 * max(1, max |x|) (a rotation keeps sizes);
bf16: the rotated values are rounded once to bf16, max |delta| <= 2e-2 and mean <= 2e-3 on N(0,1)."""

import numpy as np
import pytest
import torch

import oracle
from paper_2401_09486_b200 import binding as L
from paper_2401_09486_b200 import build, synthetic

pytestmark = pytest.mark.gpu
NOREP = L.LOMA_FLAG_NO_REP_ZONE
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _library():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    build.build_library()
    L.lib()
    torch.cuda.set_device(0)
    yield
    assert L.loma_device_status() == 0


def npf(x):
    return x.detach().to("cpu").to(torch.float64).numpy()


def check(got, want, dtype):
    d = np.abs(npf(got) - want)
    if dtype == torch.float32:
        assert d.max() <= 1e-5 * max(1.0, np.abs(want).max()), d.max()
    else:
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, (d.max(), d.mean())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("ptype", [0, 1])
@pytest.mark.parametrize("B,H,D,n,c,t,tail,flags", [(1, 1, 64, 2, 4, 4, 0, 0), (2, 3, 128, 5, 4, 16, 37, 0),
                                                    (1, 2, 128, 128, 8, 32, 0, 0),       # ids up to 32767
                                                    (2, 2, 64, 4, 1, 5, 2, 0), (1, 2, 128, 0, 4, 0, 301, 0),
                                                    (2, 2, 128, 3, 8, 32, 100, NOREP)])
def test_rope_matches_oracle(B, H, D, n, c, t, tail, flags, ptype, dtype):
    S = oracle.seq_len(n, c, t, tail, flags)
    q, k, _ = synthetic.qkv(B, H, S, D, seed=21, std=1.0, dtype=dtype)
    wq, wk = oracle.rope_apply(npf(q), npf(k), n, c, t, tail, flags, 10000.0, "contiguous" if ptype else "intermittent")
    gq, gk = q.to(DEV), k.to(DEV)
    L.loma_rope_apply(gq, gk, n, c, t, tail, flags, 0.0, ptype)
    torch.cuda.synchronize()
    check(gq, wq, dtype)
    check(gk, wk, dtype)


def test_rope_strided_views_single_tensor_and_custom_base():
    B, H, D, n, c, t = 2, 3, 128, 3, 4, 16
    S = oracle.seq_len(n, c, t)
    buf = synthetic.normal_tensor((B, S, 2, H, D), 31, 1.0, torch.float32).to(DEV)
    q, k = (buf[:, :, i].permute(0, 2, 1, 3) for i in range(2))
    q0, k0 = npf(q), npf(k)
    L.loma_rope_apply(q, None, n, c, t, 0, 0, 500000.0)
    torch.cuda.synchronize()
    wq, _ = oracle.rope_apply(q0, k0, n, c, t, theta_base=500000.0)
    check(q, wq, torch.float32)
    assert np.array_equal(npf(k), k0)          # untouched


def test_rotated_scores_see_positions_only_through_their_difference():
    """Rotating q and k on the device and taking q.k of a reading row with a memory key gives the score
    of the unrotated pair rotated by the id difference that Eq. 14 sets up (an end-to-end use of the ids)."""
    B, H, D, n, c, t = 1, 1, 128, 3, 4, 4
    S = oracle.seq_len(n, c, t)
    q, k, _ = synthetic.qkv(B, H, S, D, seed=33, dtype=torch.float32)
    gq, gk = q.to(DEV), k.to(DEV)
    L.loma_rope_apply(gq, gk, n, c, t)
    torch.cuda.synchronize()
    pos = oracle.position_ids(n, c, t)
    i, j = 2 * (2 * 16 + 4) + 3, 16 + 2                   # reading row of chunk 2, memory key of chunk 0
    got = float((gq[0, 0, i].double() * gk[0, 0, j].double()).sum())
    want = float((oracle.rope_rotate(npf(q)[0, 0, i:i + 1], np.array([pos[i] - pos[j]]))[0] * npf(k)[0, 0, j]).sum())
    assert abs(got - want) < 1e-4


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_inverse_rotation_undoes_the_rotation_and_matches_the_oracle_at_negated_positions(dtype):
    B, H, D, n, c, t, tail = 2, 2, 128, 5, 4, 16, 9
    S = oracle.seq_len(n, c, t, tail)
    q, k, _ = synthetic.qkv(B, H, S, D, seed=25, dtype=dtype)
    gq, gk = q.to(DEV), k.to(DEV)
    L.loma_rope_apply(gq, gk, n, c, t, tail, 0, 0.0, L.LOMA_ROPE_INVERSE)
    torch.cuda.synchronize()
    pos = oracle.position_ids(n, c, t, tail)
    check(gq, oracle.rope_rotate(npf(q), -pos), dtype)
    check(gk, oracle.rope_rotate(npf(k), -pos), dtype)
    L.loma_rope_apply(gq, gk, n, c, t, tail)                       # forward rotation of the inverse: back to the start
    torch.cuda.synchronize()
    tol = 1e-5 if dtype == torch.float32 else 3e-2
    assert float((gq.float().cpu() - q.float()).abs().max()) <= tol * max(1.0, float(q.float().abs().max()))


def test_differentiable_rope_then_attention_against_torch_autograd():
    """rope -> masked attention as torch ops built on the library, against torch's own autograd of the same
    composition in fp64 (rotation written with cos/sin tables from the oracle's position ids)."""
    from paper_2401_09486_b200.autograd import loma_masked_attention, loma_rope
    B, H, D, n, c, t = 1, 2, 64, 3, 2, 8
    S = oracle.seq_len(n, c, t)
    q, k, v = (x.to(DEV).requires_grad_(True) for x in synthetic.qkv(B, H, S, D, seed=27, dtype=torch.float32))
    w = synthetic.normal_tensor((B, H, S, D), 28, 1.0, torch.float32).to(DEV)
    rq, rk = loma_rope(q, k, n, c, t)
    (loma_masked_attention(rq, rk, v, n, c, t) * w).sum().backward()
    pos = torch.from_numpy(oracle.position_ids(n, c, t)).double().to(DEV)
    theta = 10000.0 ** (-2.0 * torch.arange(D // 2, dtype=torch.float64, device=DEV) / D)
    ang = pos[:, None] * theta[None, :]
    cs, sn = torch.cos(ang), torch.sin(ang)
    def rot(x):
        a, b = x[..., : D // 2], x[..., D // 2:]
        return torch.cat([a * cs - b * sn, b * cs + a * sn], dim=-1)
    q2, k2, v2 = (x.detach().double().requires_grad_(True) for x in (q, k, v))
    M = torch.from_numpy(oracle.dense_mask(n, c, t)).to(DEV)
    A = (rot(q2) @ rot(k2).transpose(-1, -2)) / D ** 0.5
    ((torch.softmax(A.masked_fill(~M, float("-inf")), dim=-1) @ v2) * w.double()).sum().backward()
    torch.cuda.synchronize()
    for g, g2 in ((q.grad, q2.grad), (k.grad, k2.grad), (v.grad, v2.grad)):
        assert float((g.double() - g2).abs().max()) <= 2e-5 * max(1.0, float(g2.abs().max()))
