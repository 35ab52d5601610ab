"""Small, self-contained launches of each kernel for profiler captures.

    python -m paper_2401_09486_b200.profile_cases decode|compress|compress_prior|masked|masked_long|bwd|bwd_long [--reps N]

Each case keeps the inputs larger than L2 (126 MB) so DRAM counters mean
something, but holds at most a few GB on the device and launches the kernel a
handful of times, so a full-counter capture ends by itself within a minute or
two.  The cases are cut-down versions of the benchmark workloads (fewer
(batch, head) pairs, same per-pair shapes).
"""

from __future__ import annotations

import argparse
import math

import torch

from . import binding as L
from . import build, synthetic


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["decode", "compress", "compress_prior", "masked", "masked_long", "bwd", "bwd_long"])
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    build.build_library()
    torch.cuda.set_device(0)
    dev = "cuda:0"
    bf = torch.bfloat16
    D = 128
    std = 1.0 / math.sqrt(D)

    if args.case in ("decode", "compress", "compress_prior"):
        B, H, c, t, mem_len = 8, 32, 4, 16, 8192          # 1/4 of the generation workload's batch: 1.08 GB of cache
        tc = c * t
        cap = mem_len + tc + t
        kc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 1, std)
        vc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 2, std)
        flags = L.LOMA_FLAG_MEM_SEES_PRIOR_MEM if args.case == "compress_prior" else 0
        ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, cap),
                             L.loma_compress_workspace_bytes(B, H, D, t, mem_len, flags)), dtype=torch.uint8, device=dev)
        if args.case == "decode":
            q, kn, vn = (x.to(dev) for x in synthetic.qkv(B, H, 1, D, 3, std, bf))
            o = torch.empty_like(q)
            for r in range(args.reps):
                L.loma_decode_attn(q, kn, vn, kc, vc, o, None, mem_len + 31 + r, ws)
        else:
            qm, km, vm = (x.to(dev) for x in synthetic.qkv(B, H, t, D, 4, std, bf))
            om = torch.empty_like(qm)
            for r in range(args.reps):
                L.loma_compress_step(qm, km, vm, kc, vc, om, None, mem_len, c, t, ws, flags)
    else:
        if args.case in ("masked", "bwd"):
            B, H, n, c, t = 1, 32, 32, 4, 16               # one batch element of the 4608-token layout: 151 MB per tensor
        else:
            B, H, n, c, t = 1, 8, 128, 8, 32               # 8 heads of the 69632-token layout: 143 MB per tensor
        S = n * (2 * c * t + t)
        q, k, v = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=bf, device=dev), 10 + i, std) for i in range(3))
        o = torch.empty_like(q)
        if args.case.startswith("bwd"):
            lse = torch.empty((B, H, S), dtype=torch.float32, device=dev)
            L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t)
            d_o = synthetic.big_normal_(torch.empty_like(q), 20, std)
            dq, dk, dv = (torch.empty_like(q) for _ in range(3))
            ws = torch.empty(L.loma_masked_attn_bwd_workspace_bytes(B, H, D, n, c, t), dtype=torch.uint8, device=dev)
            for r in range(args.reps):
                L.loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n, c, t, 0, 0, ws)
        else:
            for r in range(args.reps):
                L.loma_masked_attn_fwd(q, k, v, o, None, n, c, t)
    torch.cuda.synchronize()
    assert L.loma_device_status() == 0
    print("ok", args.case)


if __name__ == "__main__":
    main()
