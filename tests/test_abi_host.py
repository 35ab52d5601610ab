"""Host-side checks of the C-ABI library that need no GPU: it builds and loads,
exports everything include/loma.h declares, rejects bad arguments before any
CUDA call, and its host index maps agree bit for bit with the oracle."""

import ctypes
import os
import re

import numpy as np
import pytest
import torch

import oracle
from paper_2401_09486_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

INVALID, UNSUPPORTED, ALIGNMENT, CAPACITY, WORKSPACE = -1, -2, -3, -4, -5


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "loma.h")).read()
    return sorted(set(re.findall(r"LOMA_API\s+[\w\s\*]+?\b(loma_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} declared in loma.h but not exported"
        assert n in binding.SIGNATURES, f"{n} has no binding signature"
    assert sorted(binding.SIGNATURES) == names
    assert lib.loma_version() >= 100
    assert b"LOMA_OK" in lib.loma_status_string(0)
    for code in range(-7, 0):
        assert b"LOMA_ERR" in lib.loma_status_string(code)


@pytest.mark.parametrize("n,c,t,tail", [(0, 4, 0, 9), (1, 1, 1, 0), (3, 2, 2, 0), (2, 4, 4, 3), (32, 4, 16, 0),
                                        (5, 3, 7, 21), (128, 8, 32, 0), (0, 2, 3, 0)])
def test_host_layout_index_bit_exact(lib, n, c, t, tail):
    got = binding.loma_layout_index(n, c, t, tail, device="cpu")
    want = oracle.layout_index(n, c, t, tail)
    for g, w in zip(got, want):
        assert g.dtype == torch.int32
        assert np.array_equal(g.numpy(), w)


@pytest.mark.parametrize("n_tok,c,t", [(0, 4, 4), (1, 4, 4), (100, 4, 4), (257, 8, 16), (50, 3, 0), (64, 1, 5)])
def test_host_generation_index_bit_exact(lib, n_tok, c, t):
    got = binding.loma_generation_index(n_tok, c, t, device="cpu")
    want = oracle.generation_index(n_tok, c, t)
    for g, w in zip(got, want):
        assert np.array_equal(g.numpy(), w)


@pytest.mark.parametrize("n,c,t,tail", [(3, 2, 2, 0), (2, 4, 4, 3), (32, 4, 16, 5), (5, 3, 7, 21)])
def test_host_layout_index_inference_layout_bit_exact(lib, n, c, t, tail):
    f = binding.LOMA_FLAG_NO_REP_ZONE
    got = binding.loma_layout_index(n, c, t, tail, device="cpu", flags=f)
    want = oracle.layout_index(n, c, t, tail, oracle.FLAG_NO_REP_ZONE)
    for g, w in zip(got, want):
        assert np.array_equal(g.numpy(), w)


def test_layout_index_null_outputs_are_skipped(lib):
    S = oracle.seq_len(2, 2, 2)
    pos = (ctypes.c_int32 * S)()
    assert lib.loma_layout_index(2, 2, 2, 0, 0, None, None, None, None, pos, 0, None) == 0
    assert list(pos) == oracle.layout_index(2, 2, 2)[4].tolist()


def test_layout_index_rejects_bad_geometry(lib):
    buf = (ctypes.c_int32 * 64)()
    bad = [(-1, 2, 2, 0), (1, 0, 2, 0), (1, 2, -1, 0), (1, 2, 0, 0), (1, 2, 2, 5), (1, 2, 2, -1),
           (1 << 20, 64, 64, 0)]
    for n, c, t, tail in bad:
        assert lib.loma_layout_index(n, c, t, tail, 0, buf, None, None, None, None, 0, None) == INVALID


def _fwd(lib, q=0x1000, k=0x2000, v=0x3000, o=0x4000, lse=None, B=1, H=1, D=64, n=1, c=2, t=2, tc=4, tail=0,
         sb=640, sh=640, ss=64, dt=1, scale=0.0, flags=0):
    return lib.loma_masked_attn_fwd(q, k, v, o, lse, B, H, D, n, c, t, tc, tail, sb, sh, ss, dt, scale, flags,
                                    None)


def test_masked_attn_fwd_validation_precedes_any_cuda_call(lib):
    # pointers are never dereferenced: every call below must fail on the host
    assert _fwd(lib, tc=5) == INVALID                   # tc != c*t
    assert _fwd(lib, D=96) == UNSUPPORTED
    assert _fwd(lib, dt=7) == UNSUPPORTED
    assert _fwd(lib, B=-1) == INVALID
    assert _fwd(lib, q=None) == INVALID
    assert _fwd(lib, o=0x1000) == INVALID               # o aliases q
    assert _fwd(lib, q=0x1008) == ALIGNMENT
    assert _fwd(lib, ss=68, dt=1) == ALIGNMENT          # 136-byte row stride
    assert _fwd(lib, ss=32) == INVALID                  # rows overlap
    assert _fwd(lib, B=2, sb=0) == INVALID              # two batch elements on the same rows
    assert _fwd(lib, H=3, sh=0) == INVALID              # two heads on the same rows
    assert _fwd(lib, t=0, tc=0, n=1) == INVALID         # t == 0 needs n_chunks == 0
    assert _fwd(lib, tail=5) == INVALID                 # tail longer than a reading zone
    assert _fwd(lib, n=0, t=2, tc=4, tail=0) == 0       # empty sequence: no-op
    assert _fwd(lib, B=0) == 0


def test_rope_fused_steps_validation(lib):
    def dec(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, B=1, H=1, D=128, cap=8, cache_len=3, pos=3, dt=1):
        return lib.loma_decode_attn_rope(q, kn, vn, kc, vc, o, None, B, H, D, cap, cache_len, pos, 0.0, dt, 0.0, 0, None, 0, None)
    assert dec(pos=-1) == INVALID
    assert dec(kn=None, vn=None) == INVALID             # the key to rotate has to be given
    assert dec(cache_len=8) == CAPACITY
    assert dec(D=96) == UNSUPPORTED
    assert dec(q=0x1004) == ALIGNMENT
    assert dec(H=0) == 0

    def cmp_(qm=0x1000, km=0x2000, vm=0x3000, kc=0x4000, vc=0x5000, om=0x6000, B=1, H=1, D=128, cap=96, mem_len=16, c=4, t=16,
             tc=64, pos0=67, stride=4, dt=1):
        return lib.loma_compress_step_rope(qm, km, vm, kc, vc, om, None, B, H, D, cap, mem_len, c, t, tc, pos0, stride, 0.0, dt,
                                           0.0, 0, None, 0, None)
    assert cmp_(pos0=-1) == INVALID
    assert cmp_(stride=-2) == INVALID
    assert cmp_(pos0=2**31 - 10, stride=4) == INVALID    # the last id would overflow
    assert cmp_(tc=63) == INVALID
    assert cmp_(cap=79) == CAPACITY
    assert cmp_(km=None) == INVALID
    assert cmp_(B=0) == 0


def test_layer_loop_validation(lib):
    import ctypes
    arr = lambda *xs: (ctypes.c_void_p * len(xs))(*xs)
    def dec(n=2, q=arr(0x1000, 0x1100), kn=arr(0x2000, 0x2100), vn=arr(0x3000, 0x3100), kc=arr(0x4000, 0x4100),
            vc=arr(0x5000, 0x5100), o=arr(0x6000, 0x6100), B=1, H=1, D=128, cap=8, cache_len=3, dt=1):
        return lib.loma_decode_attn_layers(n, q, kn, vn, kc, vc, o, None, B, H, D, cap, cache_len, dt, 0.0, 0, None, 0, None)
    assert dec(n=-1) == INVALID
    assert dec(q=None) == INVALID
    assert dec(kc=arr(0x4000, 0x4000)) == INVALID        # two layers on one cache
    assert dec(q=arr(0x1000, 0x1104)) == ALIGNMENT       # the second layer is checked before the first is enqueued
    assert dec(kn=arr(0x2000, None)) == INVALID          # k_new without v_new in layer 1
    assert dec(cache_len=8) == CAPACITY
    assert dec(D=96) == UNSUPPORTED
    assert dec(n=0) == 0
    assert dec(H=0) == 0

    def cmp_(n=2, qm=arr(0x1000, 0x1100), km=arr(0x2000, 0x2100), vm=arr(0x3000, 0x3100), kc=arr(0x4000, 0x4100),
             vc=arr(0x5000, 0x5100), om=arr(0x6000, 0x6100), B=1, H=1, D=128, cap=96, mem_len=16, c=4, t=16, tc=64, dt=1):
        return lib.loma_compress_step_layers(n, qm, km, vm, kc, vc, om, None, B, H, D, cap, mem_len, c, t, tc, dt, 0.0, 0,
                                             None, 0, None)
    assert cmp_(tc=63) == INVALID
    assert cmp_(cap=79) == CAPACITY
    assert cmp_(km=arr(0x2000, None)) == INVALID
    assert cmp_(om=arr(0x6000, 0x6000)) == INVALID
    assert cmp_(vm=arr(0x3000, 0x3108)) == ALIGNMENT
    assert cmp_(n=0) == 0
    assert cmp_(B=0) == 0


def test_prefill_attn_validation(lib):
    def call(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, lse=None, B=1, H=1, D=128, l=4, cap=16,
             cache_len=3, dt=1, flags=0):
        return lib.loma_prefill_attn(q, kn, vn, kc, vc, o, lse, B, H, D, l, cap, cache_len, dt, 0.0, flags, None)
    assert call(cache_len=13) == CAPACITY                # 13 + 4 > 16
    assert call(l=-1) == INVALID
    assert call(kn=None) == INVALID                      # k_new without v_new
    assert call(o=0x1000) == INVALID                     # o aliases q
    assert call(q=None) == INVALID
    assert call(D=96) == UNSUPPORTED
    assert call(dt=5) == UNSUPPORTED
    assert call(vc=0x5004) == ALIGNMENT
    assert call(lse=0x7002) == ALIGNMENT
    assert call(l=0) == 0
    assert call(H=0) == 0


@pytest.mark.parametrize("l", [1, 2, 17, 64, 100, 128, 129, 200, 300, 517])
@pytest.mark.parametrize("cache_len", [0, 1, 16, 63, 64, 100, 127, 128, 500, 8192])
def test_prefill_tile_plan_reproduces_the_listing_mask(lib, l, cache_len):
    """The tensor-core kernel's plan for several tokens over a cache visits exactly the entries of
    tril(ones(l, l + k), diagonal = k) (Appendix A, `inference_input`), each once."""
    got = binding.loma_prefill_attn_plan_coverage(l, cache_len).numpy()
    want = np.tril(np.ones((l, l + cache_len), np.uint8), k=cache_len)
    assert np.array_equal(got, want), f"{int((got != want).sum())} entries differ"


def test_prefill_cache_validation(lib):
    def call(k=0x1000, v=0x2000, kc=0x3000, vc=0x4000, B=1, H=1, D=128, cap=64, n=2, c=4, t=16, tc=64, tail=3,
             sb=100000, sh=100000, ss=128, dt=1, flags=0):
        n_out = ctypes.c_int(-1)
        rc = lib.loma_prefill_cache(k, v, kc, vc, B, H, D, cap, n, c, t, tc, tail, sb, sh, ss, dt, flags,
                                    ctypes.byref(n_out), None)
        return rc, n_out.value
    assert call(cap=34)[0] == CAPACITY                  # needs 2*16 + 3 slots
    assert call(tc=60)[0] == INVALID
    assert call(k=None)[0] == INVALID
    assert call(v=0x2004)[0] == ALIGNMENT
    assert call(D=80)[0] == UNSUPPORTED
    assert call(B=0) == (0, 35)                         # nothing to do, length still reported


def test_decode_validation(lib):
    def call(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, B=1, H=1, D=128, cap=8, ln=3, dt=1,
             ws=None, wsb=0):
        return lib.loma_decode_attn(q, kn, vn, kc, vc, o, None, B, H, D, cap, ln, dt, 0.0, 0, ws, wsb, None)
    assert call(ln=8) == CAPACITY
    assert call(ln=-1) == INVALID
    assert call(D=100) == UNSUPPORTED
    assert call(kn=None) == INVALID                     # k_new and v_new must come together
    assert call(kc=None) == INVALID
    assert call(o=0x6004) == ALIGNMENT
    assert call(B=0) == 0
    # a workspace is required whenever the size query says so
    need = lib.loma_decode_workspace_bytes(32, 32, 128, 8192)
    if need:
        assert lib.loma_decode_attn(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, None, 32, 32, 128, 9000,
                                    8192, 1, 0.0, 0, None, 0, None) == WORKSPACE
        assert lib.loma_decode_attn(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, None, 32, 32, 128, 9000,
                                    8192, 1, 0.0, 0, 0x7000, need - 1, None) == WORKSPACE


def test_compress_validation(lib):
    def call(qm=0x1000, km=0x2000, vm=0x3000, kc=0x4000, vc=0x5000, om=0x6000, B=1, H=1, D=128, cap=100,
             mem_len=16, c=4, t=16, tc=64, dt=1, flags=0):
        return lib.loma_compress_step(qm, km, vm, kc, vc, om, None, B, H, D, cap, mem_len, c, t, tc, dt, 0.0,
                                      flags, None, 0, None)
    assert call(cap=79) == CAPACITY                     # needs mem_len + tc entries
    assert call(tc=63) == INVALID
    assert call(t=0, tc=0) == INVALID
    assert call(mem_len=-16) == INVALID
    assert call(D=32) == UNSUPPORTED
    assert call(vm=None) == INVALID
    assert call(vc=0x5002) == ALIGNMENT
    assert call(H=0) == 0


PLAN_GEOMS = [(3, 2, 2, 0), (2, 4, 4, 3), (5, 4, 16, 37), (9, 4, 16, 0), (3, 8, 16, 0), (3, 8, 16, 100), (3, 8, 32, 200),
              (2, 8, 32, 256), (4, 1, 5, 2), (2, 3, 7, 0), (0, 4, 0, 301), (0, 1, 0, 128), (1, 2, 64, 0), (9, 2, 8, 16),
              (2, 1, 128, 5), (2, 2, 130, 17), (2, 3, 100, 300), (3, 1, 1, 1), (17, 2, 8, 0), (2, 1, 200, 0)]


@pytest.mark.parametrize("n,c,t,tail", PLAN_GEOMS)
@pytest.mark.parametrize("flags", [0, 1, 2, 3])
def test_tensor_core_tile_plan_reproduces_the_mask_exactly(lib, n, c, t, tail, flags):
    """Every allowed (row, key) pair of Eq. 2 is visited exactly once by the
    tensor-core kernel's tile plan, and no blocked pair is visited at all."""
    got = binding.loma_masked_attn_plan_coverage(n, c, t, tail, flags).numpy()
    want = oracle.dense_mask(n, c, t, tail, flags).astype(np.uint8)
    assert got.shape == want.shape
    assert np.array_equal(got, want), f"{int((got != want).sum())} entries differ"


def test_masked_attn_bwd_validation(lib):
    def call(q=0x1000, k=0x2000, v=0x3000, o=0x4000, g=0x5000, lse=0x6000, dq=0x7000, dk=0x8000, dv=0x9000, B=1, H=1,
             D=64, n=1, c=2, t=2, tc=4, tail=0, sb=640, sh=640, ss=64, dt=1, ws=0xa000, wsb=1 << 20):
        return lib.loma_masked_attn_bwd(q, k, v, o, g, lse, dq, dk, dv, B, H, D, n, c, t, tc, tail, sb, sh, ss, dt, 0.0, 0,
                                        ws, wsb, None)
    assert call(tc=5) == INVALID
    assert call(D=96) == UNSUPPORTED
    assert call(lse=None) == INVALID
    assert call(g=None) == INVALID
    assert call(dk=0x2000) == INVALID                   # dk aliases k
    assert call(dv=0x8000) == INVALID                   # dv aliases dk
    assert call(dq=0x7008) == ALIGNMENT
    assert call(ss=68) == ALIGNMENT
    assert call(ws=None) == WORKSPACE
    assert call(wsb=8) == WORKSPACE
    assert call(ws=0xa010) == ALIGNMENT
    assert call(B=0) == 0
    need = lib.loma_masked_attn_bwd_workspace_bytes(4, 32, 128, 32, 4, 16, 0, 0)
    assert need >= 4 * 32 * 4608 * 4 and need % 256 == 0
    assert lib.loma_masked_attn_bwd_workspace_bytes(1, 1, 64, 1, 0, 2, 0, 0) == 0     # c < 1: no layout


@pytest.mark.parametrize("n,c,t,tail", PLAN_GEOMS)
@pytest.mark.parametrize("flags", [0, 1, 2, 3])
def test_key_tile_side_of_the_plan_reproduces_the_mask_exactly(lib, n, c, t, tail, flags):
    """The backward's dK/dV pass walks, per key tile, the query tiles that see it: every allowed
    (row, key) pair of Eq. 2 must again be visited exactly once and no blocked pair at all."""
    got = binding.loma_masked_attn_bwd_plan_coverage(n, c, t, tail, flags).numpy()
    want = oracle.dense_mask(n, c, t, tail, flags).astype(np.uint8)
    assert got.shape == want.shape
    assert np.array_equal(got, want), f"{int((got != want).sum())} entries differ"


def test_rope_validation(lib):
    def call(q=0x1000, k=0x2000, B=1, H=1, D=64, n=1, c=2, t=2, tc=4, tail=0, sb=640, sh=640, ss=64, dt=1, ptype=0):
        return lib.loma_rope_apply(q, k, B, H, D, n, c, t, tc, tail, sb, sh, ss, dt, 0.0, ptype, 0, None)
    assert call(tc=5) == INVALID
    assert call(ptype=4) == INVALID
    assert call(ptype=-1) == INVALID
    assert call(D=96) == UNSUPPORTED
    assert call(k=0x1000) == INVALID                    # q aliases k
    assert call(q=0x1004) == ALIGNMENT
    assert call(ss=68) == ALIGNMENT
    assert call(q=None, k=None) == 0                    # nothing to rotate
    assert call(H=0) == 0


def _random_geometries(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        c = int(rng.integers(1, 9))
        t = int(rng.choice([1, 2, 3, 5, 8, 16, 17, 32, 48, 64, 100, 128, 130, 200]))
        tc = c * t
        n = int(rng.integers(0, 7))
        tail = int(rng.integers(0, min(tc, 300) + 1))
        flags = int(rng.integers(0, 4))
        S = n * ((tc + t) if flags & 2 else (2 * tc + t)) + tail
        if 0 < S <= 2600:
            out.append((n, c, t, tail, flags))
    return out


@pytest.mark.parametrize("n,c,t,tail,flags", _random_geometries(40, 2024))
def test_both_sides_of_the_plan_on_seeded_random_geometries(lib, n, c, t, tail, flags):
    """Seeded random layouts (zone lengths on both sides of 64 and 128, odd sizes, ragged tails, every flag
    combination): the plan read by query tile and the plan read by key tile both reproduce Eq. 2 exactly."""
    want = oracle.dense_mask(n, c, t, tail, flags).astype(np.uint8)
    by_query = binding.loma_masked_attn_plan_coverage(n, c, t, tail, flags).numpy()
    by_key = binding.loma_masked_attn_bwd_plan_coverage(n, c, t, tail, flags).numpy()
    assert np.array_equal(by_query, want), f"query side: {int((by_query != want).sum())} entries differ"
    assert np.array_equal(by_key, want), f"key side: {int((by_key != want).sum())} entries differ"


def test_ragged_decode_validation(lib):
    def call(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, B=2, H=1, D=128, cap=8, lens=0x7000, mx=3,
             dt=1):
        return lib.loma_decode_attn_ragged(q, kn, vn, kc, vc, o, None, B, H, D, cap, lens, mx, dt, 0.0, 0, None, 0, None)
    assert call(mx=8) == CAPACITY
    assert call(mx=-1) == INVALID
    assert call(lens=None) == INVALID
    assert call(lens=0x7002) == ALIGNMENT
    assert call(D=100) == UNSUPPORTED
    assert call(B=0) == 0


def test_ragged_compress_validation(lib):
    def call(qm=0x1000, km=0x2000, vm=0x3000, kc=0x4000, vc=0x5000, om=0x6000, B=2, H=1, D=128, cap=100, lens=0x7000,
             mx=16, c=4, t=16, tc=64, dt=1, flags=0):
        return lib.loma_compress_step_ragged(qm, km, vm, kc, vc, om, None, B, H, D, cap, lens, mx, c, t, tc, dt, 0.0, flags,
                                             None)
    assert call(cap=79) == CAPACITY
    assert call(tc=63) == INVALID
    assert call(lens=None) == INVALID
    assert call(lens=0x7001) == ALIGNMENT
    assert call(flags=1) == UNSUPPORTED                 # prior-memory variant is not offered ragged
    assert call(D=32) == UNSUPPORTED
    assert call(B=0) == 0


def test_header_and_library_are_usable_from_plain_c(lib, tmp_path):
    """include/loma.h compiles as strict C99 and a C program linked against the library gets the documented
    answers from the entry points that need no device."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    exe = str(tmp_path / "abi_check")
    libdir = os.path.dirname(binding.library_path())
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
           os.path.join(ROOT, "tests", "c_abi", "abi_check.c"), "-o", exe, "-L", libdir, "-lloma", f"-Wl,-rpath,{libdir}"]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, out.stderr
    assert "abi_check ok" in out.stdout


def test_paged_decode_validation(lib):
    def call(q=0x1000, kn=0x2000, vn=0x3000, kp=0x4000, vp=0x5000, bt=0x6000, o=0x7000, B=2, H=1, D=128, ps=16, mp=4, npg=8,
             lens=0x8000, mx=40, dt=1):
        return lib.loma_decode_attn_paged(q, kn, vn, kp, vp, bt, o, None, B, H, D, ps, mp, npg, lens, mx, dt, 0.0, 0, None, 0,
                                          None)
    assert call(ps=24) == INVALID                       # page size must be a power of two
    assert call(mx=64) == CAPACITY                      # no slot left for the new token
    assert call(bt=None) == INVALID
    assert call(lens=None) == INVALID
    assert call(npg=0) == INVALID
    assert call(bt=0x6002) == ALIGNMENT
    assert call(D=100) == UNSUPPORTED
    assert call(B=0) == 0


def test_paged_compress_validation(lib):
    def call(qm=0x1000, km=0x2000, vm=0x3000, kp=0x4000, vp=0x5000, bt=0x6000, om=0x7000, B=2, H=1, D=128, ps=16, mp=8,
             npg=16, lens=0x8000, mx=16, c=4, t=16, tc=64, dt=1, flags=0):
        return lib.loma_compress_step_paged(qm, km, vm, kp, vp, bt, om, None, B, H, D, ps, mp, npg, lens, mx, c, t, tc, dt,
                                            0.0, flags, None)
    assert call(mx=65) == CAPACITY                      # tail would run past the table
    assert call(ps=48) == INVALID
    assert call(tc=63) == INVALID
    assert call(bt=None) == INVALID
    assert call(flags=1) == UNSUPPORTED
    assert call(lens=0x8002) == ALIGNMENT
    assert call(B=0) == 0


def test_ragged_and_paged_rope_fused_steps_validation(lib):
    """The per-sequence position arrays are checked on the host like every other pointer, after which the
    plain step's own checks apply unchanged."""
    def dec_r(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, B=2, H=1, D=128, cap=8, lens=0x7000, mx=3,
              pos=0x9000, dt=1):
        return lib.loma_decode_attn_ragged_rope(q, kn, vn, kc, vc, o, None, B, H, D, cap, lens, mx, pos, 0.0, dt, 0.0, 0, None,
                                                0, None)
    assert dec_r(pos=None) == INVALID
    assert dec_r(pos=0x9002) == ALIGNMENT
    assert dec_r(kn=None, vn=None) == INVALID           # the key to rotate has to be given
    assert dec_r(mx=8) == CAPACITY
    assert dec_r(lens=None) == INVALID
    assert dec_r(D=100) == UNSUPPORTED
    assert dec_r(B=0) == 0

    def dec_p(q=0x1000, kn=0x2000, vn=0x3000, kp=0x4000, vp=0x5000, bt=0x6000, o=0x7000, B=2, H=1, D=128, ps=16, mp=4, npg=8,
              lens=0x8000, mx=40, pos=0x9000, dt=1):
        return lib.loma_decode_attn_paged_rope(q, kn, vn, kp, vp, bt, o, None, B, H, D, ps, mp, npg, lens, mx, pos, 0.0, dt,
                                               0.0, 0, None, 0, None)
    assert dec_p(pos=None) == INVALID
    assert dec_p(pos=0x9001) == ALIGNMENT
    assert dec_p(kn=None, vn=None) == INVALID
    assert dec_p(ps=24) == INVALID
    assert dec_p(mx=64) == CAPACITY
    assert dec_p(B=0) == 0

    def cmp_r(qm=0x1000, km=0x2000, vm=0x3000, kc=0x4000, vc=0x5000, om=0x6000, B=2, H=1, D=128, cap=100, lens=0x7000,
              mx=16, c=4, t=16, tc=64, pos0s=0x9000, stride=4, dt=1, flags=0):
        return lib.loma_compress_step_ragged_rope(qm, km, vm, kc, vc, om, None, B, H, D, cap, lens, mx, c, t, tc, pos0s, stride,
                                                  0.0, dt, 0.0, flags, None)
    assert cmp_r(pos0s=None) == INVALID
    assert cmp_r(pos0s=0x9002) == ALIGNMENT
    assert cmp_r(stride=-1) == INVALID
    assert cmp_r(cap=79) == CAPACITY
    assert cmp_r(tc=63) == INVALID
    assert cmp_r(flags=1) == UNSUPPORTED
    assert cmp_r(B=0) == 0

    def cmp_p(qm=0x1000, km=0x2000, vm=0x3000, kp=0x4000, vp=0x5000, bt=0x6000, om=0x7000, B=2, H=1, D=128, ps=16, mp=8,
              npg=16, lens=0x8000, mx=16, c=4, t=16, tc=64, pos0s=0x9000, stride=4, dt=1, flags=0):
        return lib.loma_compress_step_paged_rope(qm, km, vm, kp, vp, bt, om, None, B, H, D, ps, mp, npg, lens, mx, c, t, tc,
                                                 pos0s, stride, 0.0, dt, 0.0, flags, None)
    assert cmp_p(pos0s=None) == INVALID
    assert cmp_p(pos0s=0x9003) == ALIGNMENT
    assert cmp_p(stride=-3) == INVALID
    assert cmp_p(mx=65) == CAPACITY
    assert cmp_p(ps=48) == INVALID
    assert cmp_p(B=0) == 0


def test_ragged_and_paged_prefill_validation(lib):
    def rag(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, B=2, H=1, D=128, l=4, cap=20, lens=0x7000, mx=16,
            dt=1):
        return lib.loma_prefill_attn_ragged(q, kn, vn, kc, vc, o, None, B, H, D, l, cap, lens, mx, dt, 0.0, 0, None)
    assert rag(mx=17) == CAPACITY
    assert rag(mx=-1) == INVALID
    assert rag(lens=None) == INVALID
    assert rag(lens=0x7002) == ALIGNMENT
    assert rag(kn=None) == INVALID                       # k_new without v_new
    assert rag(o=0x1000) == INVALID                      # o aliases q
    assert rag(D=96) == UNSUPPORTED
    assert rag(l=0) == 0 and rag(B=0) == 0

    def pag(q=0x1000, kn=0x2000, vn=0x3000, kp=0x4000, vp=0x5000, bt=0x6000, o=0x7000, B=2, H=1, D=128, l=4, ps=16, mp=2,
            npg=8, lens=0x8000, mx=28, dt=1):
        return lib.loma_prefill_attn_paged(q, kn, vn, kp, vp, bt, o, None, B, H, D, l, ps, mp, npg, lens, mx, dt, 0.0, 0, None)
    assert pag(mx=29) == CAPACITY                        # the new rows would run past the table
    assert pag(ps=24) == INVALID
    assert pag(bt=None) == INVALID
    assert pag(lens=None) == INVALID
    assert pag(npg=0) == INVALID
    assert pag(bt=0x6002) == ALIGNMENT
    assert pag(dt=7) == UNSUPPORTED
    assert pag(l=0) == 0


def test_rope_fused_prompt_piece_validation(lib):
    def uni(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, B=2, H=1, D=128, l=4, cap=20, cache_len=16,
            pos0=100, dt=1):
        return lib.loma_prefill_attn_rope(q, kn, vn, kc, vc, o, None, B, H, D, l, cap, cache_len, pos0, 0.0, dt, 0.0, 0, None)
    assert uni(pos0=-1) == INVALID
    assert uni(pos0=2**31 - 2) == INVALID                # the last id would overflow
    assert uni(kn=None, vn=None) == INVALID              # the keys to rotate have to be given
    assert uni(cache_len=17) == CAPACITY
    assert uni(D=96) == UNSUPPORTED
    assert uni(o=0x1000) == INVALID
    assert uni(l=0) == 0

    def rag(q=0x1000, kn=0x2000, vn=0x3000, kc=0x4000, vc=0x5000, o=0x6000, B=2, H=1, D=128, l=4, cap=20, lens=0x7000, mx=16,
            pos=0x9000, dt=1):
        return lib.loma_prefill_attn_ragged_rope(q, kn, vn, kc, vc, o, None, B, H, D, l, cap, lens, mx, pos, 0.0, dt, 0.0, 0,
                                                 None)
    assert rag(pos=None) == INVALID
    assert rag(pos=0x9002) == ALIGNMENT
    assert rag(lens=None) == INVALID
    assert rag(mx=17) == CAPACITY
    assert rag(B=0) == 0

    def pag(q=0x1000, kn=0x2000, vn=0x3000, kp=0x4000, vp=0x5000, bt=0x6000, o=0x7000, B=2, H=1, D=128, l=4, ps=16, mp=2,
            npg=8, lens=0x8000, mx=28, pos=0x9000, dt=1):
        return lib.loma_prefill_attn_paged_rope(q, kn, vn, kp, vp, bt, o, None, B, H, D, l, ps, mp, npg, lens, mx, pos, 0.0,
                                                dt, 0.0, 0, None)
    assert pag(pos=None) == INVALID
    assert pag(mx=29) == CAPACITY
    assert pag(ps=24) == INVALID
    assert pag(bt=None) == INVALID
    assert pag(l=0) == 0
