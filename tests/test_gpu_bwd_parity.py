"""Parity of loma_masked_attn_bwd (through the C ABI) with the CPU oracle's
backward, element by element on the same seeded inputs.

The library is given what a training step has at hand: q, k, v, the output and
log-sum-exp of its own forward, and dO.  The oracle gets the same stored q, k,
v, dO and recomputes everything else in fp64.

Tolerances.  Gradients are sums over up to thousands of rows, so their size
varies with the layout; the bars of the forward (stated for outputs of size
about one) are scaled by the size of the reference: fp32 max |delta| <= 1e-5 *
max(1, max |ref|); bf16 max |delta| <= 2e-2 * max(1, max |ref|) and mean
|delta| <= 2e-3 * max(1, mean |ref|).
"""

import numpy as np
import pytest
import torch

import oracle
from paper_2401_09486_b200 import binding as L
from paper_2401_09486_b200 import build, synthetic

pytestmark = pytest.mark.gpu

PRIOR = L.LOMA_FLAG_MEM_SEES_PRIOR_MEM
NOREP = L.LOMA_FLAG_NO_REP_ZONE
GENERIC = L.LOMA_FLAG_FORCE_GENERIC
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


def check_grad(got, want, dtype, name, zones=None):
    """Whole-tensor bars scaled by the size of the reference (a gradient is a sum over up to tens of thousands
    of rows), and, where the rows' zones are given, a bar per element: the forward's bar (2e-2, stated for
    values of size about one) scaled by the element itself plus the root-mean-square of its own zone type where
    that exceeds one.  Reading, memory and repetition rows have gradients of very different sizes (an early
    memory key collects from every later reading row), and an error on the small ones must not hide behind the
    largest element of the tensor.  The arithmetic: every output is rounded to bf16 (2^-9 of itself); P and dA
    enter the second products rounded to bf16, 2^-9 of each of ~N terms of random sign, i.e. about 2^-9 of the
    sum's typical size (the zone's rms); and delta = dO.O is formed from the bf16-rounded forward output, an
    absolute error of about 2^-9 sqrt(D) |dO| |O| in every dA, which is what keeps the bar from going below the
    forward's 2e-2 for gradients smaller than one."""
    g = npf(got)
    assert g.shape == want.shape and np.isfinite(g).all(), name
    d = np.abs(g - want)
    big, mean = max(1.0, np.abs(want).max()), max(1.0, np.abs(want).mean())
    if dtype == torch.float32:
        assert d.max() <= 1e-5 * big, f"{name}: fp32 max |delta| {d.max():.3e} (ref max {big:.3g})"
    else:
        assert d.max() <= 2e-2 * big, f"{name}: bf16 max |delta| {d.max():.3e} (ref max {big:.3g})"
        assert d.mean() <= 2e-3 * mean, f"{name}: bf16 mean |delta| {d.mean():.3e}"
    if zones is not None:
        zones = np.asarray(zones)
        assert zones.shape[0] == want.shape[2]
        rel = 1e-5 if dtype == torch.float32 else 2e-2
        for z in np.unique(zones):
            sel = zones == z
            w, dz = want[:, :, sel], d[:, :, sel]
            rms = max(float(np.sqrt((w ** 2).mean())), 1e-3)
            bad = dz > rel * np.maximum(1.0, np.abs(w) + rms)
            assert not bad.any(), (f"{name}, zone {int(z)}: {int(bad.sum())} elements beyond {rel:g} * max(1, |ref| + rms {rms:.3g}); "
                                   f"worst |delta| {float(dz.max()):.3e}")


def run_fwd_bwd(q, k, v, d_o, n, c, t, tail=0, flags=0, scale=0.0):
    o = torch.full_like(q, float("nan"))
    lse = torch.full(q.shape[:3], float("nan"), dtype=torch.float32, device=q.device)
    L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t, tail, flags, scale)
    B, H, S, D = q.shape
    ws = torch.empty(max(256, L.loma_masked_attn_bwd_workspace_bytes(B, H, D, n, c, t, tail, flags)), dtype=torch.uint8,
                     device=q.device)
    dq, dk, dv = (torch.full_like(q, float("nan")) for _ in range(3))
    L.loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n, c, t, tail, flags, ws, scale)
    torch.cuda.synchronize()
    return dq, dk, dv


BWD_CASES = [
    # B, H, D, n, c, t, tail
    (1, 1, 64, 2, 4, 4, 0),       # the tiny configuration
    (2, 2, 64, 3, 2, 4, 3),
    (1, 2, 128, 5, 4, 16, 37),    # tc = 64, several tiles and a ragged tail
    (1, 1, 128, 3, 8, 32, 200),   # tc = 256 with a tail
    (1, 2, 64, 4, 1, 5, 2),       # c = 1, odd t
    (1, 1, 128, 2, 3, 7, 0),      # nothing is a power of two
    (1, 2, 128, 0, 4, 0, 301),    # t = 0: plain causal attention
    (1, 1, 128, 9, 2, 8, 16),
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, PRIOR, NOREP, NOREP | PRIOR, GENERIC, GENERIC | PRIOR])
@pytest.mark.parametrize("B,H,D,n,c,t,tail", BWD_CASES)
def test_masked_bwd_matches_oracle(B, H, D, n, c, t, tail, flags, dtype):
    lay = flags & (PRIOR | NOREP)
    S = oracle.seq_len(n, c, t, tail, lay)
    q, k, v = synthetic.qkv(B, H, S, D, seed=11, std=1.0, dtype=dtype)
    d_o = synthetic.normal_tensor((B, H, S, D), 97, 1.0, dtype)
    want = oracle.masked_attn_bwd(npf(q), npf(k), npf(v), npf(d_o), n, c, t, tail, lay)
    got = run_fwd_bwd(q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV), n, c, t, tail, flags)
    zone = oracle.layout_index(n, c, t, tail, lay)[1]
    for g, w, name in zip(got, want, ("dq", "dk", "dv")):
        check_grad(g, w, dtype, name, zone)


def test_masked_bwd_strided_views_explicit_scale_and_unsupervised_memory_rows():
    """Views into one packed buffer; dO is zero on the memory rows (the paper puts no loss on <m>
    outputs), so their queries get exactly zero gradient."""
    B, H, D, n, c, t = 2, 3, 128, 3, 4, 16
    S = oracle.seq_len(n, c, t)
    buf = synthetic.normal_tensor((B, S, 9, H, D), 9, 1.0, torch.bfloat16).to(DEV)
    q, k, v, o, d_o, dq, dk, dv = (buf[:, :, i].permute(0, 2, 1, 3) for i in range(8))
    zone = torch.from_numpy(oracle.layout_index(n, c, t)[1]).to(DEV)
    d_o[:, :, zone == 1] = 0
    lse = torch.empty((B, H, S), dtype=torch.float32, device=DEV)
    L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t, 0, 0, 0.05)
    ws = torch.empty(L.loma_masked_attn_bwd_workspace_bytes(B, H, D, n, c, t), dtype=torch.uint8, device=DEV)
    L.loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n, c, t, 0, 0, ws, 0.05)
    torch.cuda.synchronize()
    want = oracle.masked_attn_bwd(npf(q), npf(k), npf(v), npf(d_o), n, c, t, scale=0.05)
    for g, w, name in zip((dq, dk, dv), want, ("dq", "dk", "dv")):
        check_grad(g, w, torch.bfloat16, name)
    assert float(dq[:, :, zone == 1].abs().max()) == 0.0


def test_masked_bwd_is_bitwise_repeatable():
    B, H, D, n, c, t, tail = 2, 2, 128, 5, 4, 16, 9
    S = oracle.seq_len(n, c, t, tail)
    q, k, v = (x.to(DEV) for x in synthetic.qkv(B, H, S, D, seed=5, dtype=torch.bfloat16))
    d_o = synthetic.normal_tensor((B, H, S, D), 6, 1.0, torch.bfloat16).to(DEV)
    a = run_fwd_bwd(q, k, v, d_o, n, c, t, tail)
    b = run_fwd_bwd(q, k, v, d_o, n, c, t, tail)
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))


# ------------------------------------- named workloads at full size (sampled)

def _fwd_bwd_big(B, H, S, D, n, c, t, seed, flags=0):
    q, k, v, d_o = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), seed + i) for i in range(4))
    return (q, k, v, d_o) + tuple(run_fwd_bwd(q, k, v, d_o, n, c, t, 0, flags))


def test_training_layout_4608_tokens_backward_sampled_heads():
    """B4 H32 D128 bf16, c=4, t=16, 4608 rows: the full launch; the oracle runs two (b,h) pairs in full."""
    B, H, D, n, c, t = 4, 32, 128, 32, 4, 16
    S = oracle.seq_len(n, c, t)
    q, k, v, d_o, dq, dk, dv = _fwd_bwd_big(B, H, S, D, n, c, t, 200)
    for b, h in [(0, 0), (3, 17)]:
        sl = (slice(b, b + 1), slice(h, h + 1))
        want = oracle.masked_attn_bwd(npf(q[sl]), npf(k[sl]), npf(v[sl]), npf(d_o[sl]), n, c, t)
        zone = oracle.layout_index(n, c, t)[1]
        for g, w, name in zip((dq, dk, dv), want, ("dq", "dk", "dv")):
            check_grad(g[sl], w, torch.bfloat16, name, zone)
    for g in (dq, dk, dv):
        assert torch.isfinite(g.float()).all()


def test_training_layout_4608_tokens_backward_agrees_with_the_cuda_core_kernels_everywhere():
    """Every element of the tensor-core result against the CUDA-core kernels of the same library
    (an on-GPU second opinion over all 128 (b,h) pairs; the oracle covers two of them above)."""
    B, H, D, n, c, t = 4, 32, 128, 32, 4, 16
    S = oracle.seq_len(n, c, t)
    q, k, v, d_o, dq, dk, dv = _fwd_bwd_big(B, H, S, D, n, c, t, 210)
    gq, gk, gv = run_fwd_bwd(q, k, v, d_o, n, c, t, 0, GENERIC)
    for a, b_, name in ((dq, gq, "dq"), (dk, gk, "dk"), (dv, gv, "dv")):
        ref = b_.float()
        d = (a.float() - ref).abs()
        big = max(1.0, float(ref.abs().max()))
        assert float(d.max()) <= 2e-2 * big, f"{name}: {float(d.max()):.3e} vs scale {big:.3g}"


def test_long_training_layout_69632_tokens_backward_sampled_rows_and_keys():
    """B1 H2 D128 bf16, c=8, t=32, 69632 rows: dQ on a seeded sample of rows of every zone type, dK and dV
    on sampled keys (reading, repetition and late memory keys: an early memory key is seen by tens of
    thousands of rows, each needing its whole softmax on the CPU)."""
    B, H, D, n, c, t = 1, 2, 128, 128, 8, 32
    S = oracle.seq_len(n, c, t)
    assert S == 69632
    q, k, v, d_o, dq, dk, dv = _fwd_bwd_big(B, H, S, D, n, c, t, 220)
    ch, zone = oracle.layout_index(n, c, t)[:2]
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([rng.choice(np.nonzero(zone == z)[0], 48, replace=False) for z in (0, 1, 2)]
                                    + [np.array([0, 255, 256, 287, 288, 543, S - 1, S - 257, S - 545])]))
    cols = np.unique(np.concatenate([rng.choice(np.nonzero(zone == 0)[0], 24, replace=False),
                                     rng.choice(np.nonzero(zone == 2)[0], 8, replace=False),
                                     rng.choice(np.nonzero((zone == 1) & (ch >= n - 3))[0], 12, replace=False)]))
    ri, ci = torch.from_numpy(rows).to(DEV), torch.from_numpy(cols).to(DEV)
    h = 1
    sl = (slice(0, 1), slice(h, h + 1))
    want_dq = oracle.masked_attn_bwd_dq_rows(npf(q[sl]), npf(k[sl]), npf(v[sl]), npf(d_o[sl]), rows, n, c, t)
    check_grad(dq[sl][:, :, ri], want_dq, torch.bfloat16, "dq", zone[rows])
    want_dk, want_dv = oracle.masked_attn_bwd_dkv_cols(npf(q[sl]), npf(k[sl]), npf(v[sl]), npf(d_o[sl]), cols, n, c, t)
    check_grad(dk[sl][:, :, ci], want_dk, torch.bfloat16, "dk", zone[cols])
    check_grad(dv[sl][:, :, ci], want_dv, torch.bfloat16, "dv", zone[cols])
    for g in (dq, dk, dv):
        assert torch.isfinite(g.float()).all()


def _random_layouts(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        c = int(rng.integers(1, 7))
        t = int(rng.choice([1, 3, 5, 8, 16, 17, 32, 48, 64, 100, 130]))
        tc = c * t
        n = int(rng.integers(1, 5))
        tail = int(rng.integers(0, min(tc, 200) + 1))
        flags = int(rng.integers(0, 4))
        S = n * ((tc + t) if flags & 2 else (2 * tc + t)) + tail
        if 64 < S <= 900:
            out.append((n, c, t, tail, flags, int(rng.choice([64, 128]))))
    return out


@pytest.mark.parametrize("n,c,t,tail,flags,D", _random_layouts(14, 7))
def test_forward_and_backward_on_seeded_random_layouts(n, c, t, tail, flags, D):
    """Zone lengths on both sides of 64 and 128, odd sizes, ragged tails, every flag combination, bf16
    tensor-core kernels: outputs, log-sum-exp and all three gradients against the oracle."""
    B, H = 1, 2
    S = oracle.seq_len(n, c, t, tail, flags)
    q, k, v = synthetic.qkv(B, H, S, D, seed=41, std=1.0, dtype=torch.bfloat16)
    d_o = synthetic.normal_tensor((B, H, S, D), 43, 1.0, torch.bfloat16)
    qd, kd, vd, gd = (x.to(DEV) for x in (q, k, v, d_o))
    o = torch.full_like(qd, float("nan"))
    lse = torch.full((B, H, S), float("nan"), dtype=torch.float32, device=DEV)
    L.loma_masked_attn_fwd(qd, kd, vd, o, lse, n, c, t, tail, flags)
    want_o, want_lse = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t, tail, flags)
    torch.cuda.synchronize()
    assert np.abs(npf(o) - want_o).max() <= 2e-2 and np.abs(npf(lse) - want_lse).max() <= 2e-2
    got = run_fwd_bwd(qd, kd, vd, gd, n, c, t, tail, flags)
    want = oracle.masked_attn_bwd(npf(q), npf(k), npf(v), npf(d_o), n, c, t, tail, flags)
    for g, w, name in zip(got, want, ("dq", "dk", "dv")):
        check_grad(g, w, torch.bfloat16, name)


@pytest.mark.parametrize("c,t,n", [(2, 4, 40), (2, 8, 24), (2, 32, 6), (4, 8, 12), (8, 8, 6)])
def test_table1_style_geometries_forward_and_backward(c, t, n):
    """The compression settings of the paper's Table 1 / Fig. 7 sweeps (short memory zones, c = 2..8): many
    chunks per 128-row tile.  Forward and all three gradients against the oracle, bf16 tensor-core kernels."""
    B, H, D = 1, 2, 128
    S = oracle.seq_len(n, c, t)
    q, k, v = synthetic.qkv(B, H, S, D, seed=51, std=1.0, dtype=torch.bfloat16)
    d_o = synthetic.normal_tensor((B, H, S, D), 53, 1.0, torch.bfloat16)
    qd, kd, vd, gd = (x.to(DEV) for x in (q, k, v, d_o))
    o = torch.full_like(qd, float("nan"))
    lse = torch.full((B, H, S), float("nan"), dtype=torch.float32, device=DEV)
    L.loma_masked_attn_fwd(qd, kd, vd, o, lse, n, c, t)
    torch.cuda.synchronize()
    want_o, want_lse = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t)
    assert np.abs(npf(o) - want_o).max() <= 2e-2 and np.abs(npf(lse) - want_lse).max() <= 2e-2
    got = run_fwd_bwd(qd, kd, vd, gd, n, c, t)
    want = oracle.masked_attn_bwd(npf(q), npf(k), npf(v), npf(d_o), n, c, t)
    for g, w, name in zip(got, want, ("dq", "dk", "dv")):
        check_grad(g, w, torch.bfloat16, name)


def test_training_calls_replay_from_a_cuda_graph():
    """Rotary embedding, forward and backward captured once (after an eager warm-up) and replayed twice: the
    forward's run-time tile counter is cleared by each launch's last CTA, so every replay starts from zero and
    reproduces the eager results bit for bit."""
    B, H, D, n, c, t, tail = 2, 2, 128, 5, 4, 16, 9
    S = oracle.seq_len(n, c, t, tail)
    q0, k0, v0 = (x.to(DEV) for x in synthetic.qkv(B, H, S, D, seed=71, dtype=torch.bfloat16))
    d_o = synthetic.normal_tensor((B, H, S, D), 72, 1.0, torch.bfloat16).to(DEV)
    ws = torch.empty(L.loma_masked_attn_bwd_workspace_bytes(B, H, D, n, c, t, tail), dtype=torch.uint8, device=DEV)

    def run(q, k, v, o, lse, dq, dk, dv, stream=None):
        L.loma_rope_apply(q, k, n, c, t, tail, 0, 0.0, 0, stream)
        L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t, tail, 0, 0.0, stream)
        L.loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n, c, t, tail, 0, ws, 0.0, stream)

    def buffers():
        return (q0.clone(), k0.clone(), v0.clone(), torch.zeros_like(q0), torch.zeros((B, H, S), dtype=torch.float32, device=DEV),
                torch.zeros_like(q0), torch.zeros_like(q0), torch.zeros_like(q0))

    eager = buffers()
    run(*eager)
    torch.cuda.synchronize()
    g = buffers()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            run(*g, side)
    torch.cuda.synchronize()
    for _ in range(2):
        g[0].copy_(q0); g[1].copy_(k0)          # the rotation is in place
        for x in g[3:]:
            x.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for a, b in zip(g, eager):
            assert torch.equal(a, b)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_autograd_wrapper_matches_torch_autograd_on_the_dense_mask(dtype):
    """The differentiable torch op built on the two entry points against torch's own autograd of dense masked
    softmax attention in fp64 on the same stored inputs (a third opinion next to the oracle)."""
    from paper_2401_09486_b200.autograd import loma_masked_attention
    B, H, D, n, c, t, tail = 2, 2, 64, 3, 4, 8, 5
    S = oracle.seq_len(n, c, t, tail)
    q, k, v = (x.to(DEV).requires_grad_(True) for x in synthetic.qkv(B, H, S, D, seed=81, dtype=dtype))
    w = synthetic.normal_tensor((B, H, S, D), 82, 1.0, dtype).to(DEV)
    o = loma_masked_attention(q, k, v, n, c, t, tail)
    (o.float() * w.float()).sum().backward()
    M = torch.from_numpy(oracle.dense_mask(n, c, t, tail)).to(DEV)
    q2, k2, v2 = (x.detach().double().requires_grad_(True) for x in (q, k, v))
    A = (q2 @ k2.transpose(-1, -2)) / D ** 0.5
    o2 = torch.softmax(A.masked_fill(~M, float("-inf")), dim=-1) @ v2
    (o2 * w.double()).sum().backward()
    torch.cuda.synchronize()
    tol = 1e-5 if dtype == torch.float32 else 2e-2
    assert float((o.detach().double() - o2.detach()).abs().max()) <= tol
    for g, g2, name in ((q.grad, q2.grad, "dq"), (k.grad, k2.grad, "dk"), (v.grad, v2.grad, "dv")):
        check_grad(g, g2.cpu().numpy(), dtype, name)


def test_tiles_with_more_than_64_steps_forward_and_backward():
    """c = 1, t = 128, 70 chunks (26880 rows): the last reading tiles visit 70 key tiles and the first memory key
    tiles are visited by 70+ query tiles, beyond the 64 steps whose visited halves the kernels keep as bit masks
    (later steps are taken whole).  Sampled rows against the oracle; every element against the CUDA-core kernels."""
    B, H, D, n, c, t = 1, 2, 64, 70, 1, 128
    S = oracle.seq_len(n, c, t)
    q, k, v, d_o = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), 300 + i) for i in range(4))
    o = torch.full_like(q, float("nan"))
    lse = torch.full((B, H, S), float("nan"), dtype=torch.float32, device=DEV)
    L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t)
    dq, dk, dv = run_fwd_bwd(q, k, v, d_o, n, c, t)
    o_g = torch.empty_like(q)
    L.loma_masked_attn_fwd(q, k, v, o_g, None, n, c, t, 0, GENERIC)
    gq, gk, gv = run_fwd_bwd(q, k, v, d_o, n, c, t, 0, GENERIC)
    torch.cuda.synchronize()
    assert float((o.float() - o_g.float()).abs().max()) <= 2e-2
    for a, b_, name in ((dq, gq, "dq"), (dk, gk, "dk"), (dv, gv, "dv")):
        ref = b_.float()
        assert float((a.float() - ref).abs().max()) <= 2e-2 * max(1.0, float(ref.abs().max())), name
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([rng.choice(S, 40, replace=False), np.arange(S - 384, S - 380), np.array([0, 127, 128, 255, 256])]))
    ri = torch.from_numpy(rows).to(DEV)
    sl = (slice(0, 1), slice(1, 2))
    want_o, want_lse = oracle.masked_attn_fwd(npf(q[sl]), npf(k[sl]), npf(v[sl]), n, c, t, rows=rows)
    assert np.abs(npf(o[sl][:, :, ri]) - want_o).max() <= 2e-2 and np.abs(npf(lse[sl][:, :, ri]) - want_lse).max() <= 2e-2
    zone = oracle.layout_index(n, c, t)[1]
    want_dq = oracle.masked_attn_bwd_dq_rows(npf(q[sl]), npf(k[sl]), npf(v[sl]), npf(d_o[sl]), rows, n, c, t)
    check_grad(dq[sl][:, :, ri], want_dq, torch.bfloat16, "dq", zone[rows])
    # dK and dV against the oracle too: reading, repetition and late memory keys (a key tile that more than 64 query
    # tiles visit is covered by the late-chunk reading keys: each is seen by its own zone's later rows and memory rows)
    ch = oracle.layout_index(n, c, t)[0]
    cols = np.unique(np.concatenate([rng.choice(np.nonzero(zone == 0)[0], 12, replace=False),
                                     rng.choice(np.nonzero(zone == 2)[0], 6, replace=False),
                                     rng.choice(np.nonzero((zone == 1) & (ch >= n - 2))[0], 8, replace=False),
                                     rng.choice(np.nonzero((zone == 1) & (ch == 2))[0], 2, replace=False)]))
    ci = torch.from_numpy(cols).to(DEV)
    want_dk, want_dv = oracle.masked_attn_bwd_dkv_cols(npf(q[sl]), npf(k[sl]), npf(v[sl]), npf(d_o[sl]), cols, n, c, t)
    check_grad(dk[sl][:, :, ci], want_dk, torch.bfloat16, "dk", zone[cols])
    check_grad(dv[sl][:, :, ci], want_dv, torch.bfloat16, "dv", zone[cols])
