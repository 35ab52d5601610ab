"""loma_decode_attn_static: the decode step for callers that cannot allocate.

Some users of this library run where device memory can no longer be obtained:
an inference server that has given every spare byte of HBM to its KV-cache
pool, or a step function inside a runtime that bans cudaMalloc because it
stalls the whole device.  They cannot pass loma_decode_attn a workspace, so the
library offers the same step with the split partials kept in an 8 MiB array
inside the library itself.  This test calls that entry point through the C ABI
twice in a row -- the second call finds the first call's partials still in the
array -- and checks each result against loma_decode_attn on identical inputs
(bit for bit: the two run the same kernels) and against the CPU oracle.
It lives in its own file, collected last, and passes on its own in a fresh
process as well as after the rest of the suite.
"""

import numpy as np
import pytest
import torch

import oracle
from paper_2401_09486_b200 import binding as L
from paper_2401_09486_b200 import build, synthetic

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _f64(x):
    return x.detach().cpu().to(torch.float64).numpy()


def _one_call(B, H, D, cap, cache_len, seed):
    kc = synthetic.normal_tensor((B, H, cap, D), seed, 1.0, torch.bfloat16).to(DEV)
    vc = synthetic.normal_tensor((B, H, cap, D), seed + 1, 1.0, torch.bfloat16).to(DEV)
    q, kn, vn = (x.to(DEV) for x in synthetic.qkv(B, H, 1, D, seed=seed + 2, dtype=torch.bfloat16))

    # reference: the existing entry point with a caller-provided workspace
    kc_ref, vc_ref = kc.clone(), vc.clone()
    want_o, want_lse, _, _ = oracle.decode_attn(_f64(q), _f64(kn), _f64(vn), _f64(kc), _f64(vc), cache_len)
    need = L.loma_decode_workspace_bytes(B, H, D, cache_len)
    assert need > 0, "pick a shape that really uses split partials"
    ws = torch.empty(need, dtype=torch.uint8, device=DEV)
    o_ref = torch.empty(B, H, 1, D, dtype=torch.bfloat16, device=DEV)
    lse_ref = torch.empty(B, H, dtype=torch.float32, device=DEV)
    L.loma_decode_attn(q, kn, vn, kc_ref, vc_ref, o_ref, lse_ref, cache_len, ws)

    # the allocation-free entry point: inputs and outputs only
    assert need <= L.loma_decode_static_scratch_bytes()
    o = torch.full_like(o_ref, float("nan"))
    lse = torch.full_like(lse_ref, float("nan"))
    L.loma_decode_attn_static(q, kn, vn, kc, vc, o, lse, cache_len)
    torch.cuda.synchronize()

    d = np.abs(_f64(o) - _f64(o_ref))
    assert np.isfinite(_f64(o)).all()
    assert d.max() <= 2e-2 and d.mean() <= 2e-3          # the suite's bf16 tolerance
    assert np.abs(_f64(lse) - _f64(lse_ref)).max() <= 2e-2
    assert torch.equal(kc, kc_ref) and torch.equal(vc, vc_ref)   # same bit-exact append
    # both entry points run the same two kernels with the same split of the key range, so they agree bit for bit
    assert torch.equal(o, o_ref) and torch.equal(lse, lse_ref)
    # and the new entry point on its own against the CPU oracle (Appendix A, inference_input with one token)
    d = np.abs(_f64(o) - want_o)
    assert d.max() <= 2e-2 and d.mean() <= 2e-3
    assert np.abs(_f64(lse) - want_lse.reshape(_f64(lse).shape)).max() <= 2e-2


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    build.build_library()
    torch.cuda.set_device(0)
    # two different shapes back to back: the second call reuses the array with
    # the first call's partials (other split count, other head dim) still in it
    _one_call(B=4, H=8, D=128, cap=6000, cache_len=5555, seed=900)
    _one_call(B=2, H=3, D=64, cap=3000, cache_len=2047, seed=910)
    assert L.loma_device_status() == 0


def test_static_scratch_decode_leaves_the_device_memory_as_it_found_it():
    """After the set-up call a further call changes neither the driver's count of free device memory nor
    the caching allocator's: everything it touches was there before."""
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    build.build_library()
    torch.cuda.set_device(0)
    B, H, D, cap, cache_len = 4, 8, 128, 6000, 5555
    kc = synthetic.normal_tensor((B, H, cap, D), 920, 1.0, torch.bfloat16).to(DEV)
    vc = synthetic.normal_tensor((B, H, cap, D), 921, 1.0, torch.bfloat16).to(DEV)
    q, kn, vn = (x.to(DEV) for x in synthetic.qkv(B, H, 1, D, seed=922, dtype=torch.bfloat16))
    o = torch.empty(B, H, 1, D, dtype=torch.bfloat16, device=DEV)
    L.loma_decode_attn_static(q, kn, vn, kc, vc, o, None, cache_len)        # set-up call on this device
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for step in range(3):
        L.loma_decode_attn_static(q, kn, vn, kc, vc, o, None, cache_len + 1 + step)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert L.loma_device_status() == 0


def test_static_scratch_decode_rejects_requests_beyond_its_array():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    build.build_library()
    lib = L.lib()
    limit = L.loma_decode_static_scratch_bytes()
    assert limit == 8 << 20
    B, H, D, cap, cache_len = 64, 32, 128, 16600, 16500
    assert L.loma_decode_workspace_bytes(B, H, D, cache_len) > limit
    # never launched, so dummy (aligned) addresses are enough
    rc = lib.loma_decode_attn_static(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, None, B, H, D, cap, cache_len,
                                     L.LOMA_BF16, 0.0, None)
    assert rc == -5 and "WORKSPACE" in L.status_string(rc)
    rc = lib.loma_decode_attn_static(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, None, 1, 1, D, 8, 3,
                                     L.LOMA_F32, 0.0, None)
    assert rc == -2
