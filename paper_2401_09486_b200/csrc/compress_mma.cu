// Compress step for bf16: the t <m> queries of one (batch, head) over the
// uncompressed tail and their own keys (Section 3.1 step 2, all-ones mask of
// Appendix A), fused with the in-place compaction of the cache (step 3).
//
// With t = 16 query rows per key row the step has ~16 flop per byte: it is bound
// by HBM (the short default variant by the latency of one CTA's chain of loads
// and phases: it has a kernel of its own further down, compress_one_stage_kernel),
// but too heavy for the CUDA cores when the prior-memory variant streams the whole cache.  The
// 16 queries are exactly one M = 16 tile of the warp-level tensor-core
// instruction (mma.sync.m16n8k16); the 128-row tcgen05 tile would idle 7/8 of
// the array here, so this kernel uses the warp-level path on purpose.
//
//   Memory zones longer than 16 take several 16-row query tiles, each its own CTA.
//   CTA (4 warps) = one key range of one (b,h) (and one query tile).  The last range of a (b,h) is
//   always [tail (tc rows) ; k_mem (t rows)]; with the prior-memory flag the
//   earlier ranges cut cache[0, mem_len) into pieces.
//   K and V rows are staged 64 at a time in shared memory with 16-byte
//   cp.async copies (double buffered), padded rows so ldmatrix is conflict free.
//   Each warp takes 16 of the 64 staged keys: S = Q K^T (16 x 16), online
//   softmax in registers, O += P V with P straight from the accumulator
//   registers.  Warps are merged in shared memory; ranges through the workspace
//   and a small merge kernel (fixed order: bitwise repeatable).
//   Compaction (t <= 16; longer zones compact in a second, stream-ordered launch because several
//   CTAs then read the same tail): the CTA that owns the tail is the only reader of the slots
//   [mem_len, mem_len + t) in this launch; after a block barrier it overwrites
//   them with k_mem / v_mem using 16-byte vector stores.
#include <math.h>

#include "loma_internal.cuh"

namespace loma {

constexpr int CMP_WARPS = 4;
constexpr int CMP_CHUNK = 64;          // keys staged per pipeline stage
constexpr int CMP_PRIOR_LEN = 1024;    // keys per prior-memory range (when there are many (b,h))

int compress_num_prior(int BH, int mem_len, unsigned flags) {
    if (!(flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM) || mem_len <= 0) return 0;
    int by_len = (mem_len + CMP_PRIOR_LEN - 1) / CMP_PRIOR_LEN;
    int by_fill = (4 * 148 + BH - 1) / BH - 1;
    int n = by_len > by_fill ? by_len : by_fill;
    int cap = (mem_len + 255) / 256;
    if (n > cap) n = cap;
    if (n > 255) n = 255;
    if (n < 1) n = 1;
    return n;
}

size_t compress_workspace_bytes(int BH, int D, int t, int mem_len, unsigned flags) {
    if (t > 128) return 0;   // handled by the CUDA-core kernel, which needs none
    const int np = compress_num_prior(BH, mem_len, flags);
    if (np == 0) return 0;
    const int mt = (t + 15) / 16;
    return (size_t)BH * (np + 1) * mt * 16 * (D + 2) * sizeof(float);
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;   // 0 source bytes = zero fill
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int D>
struct CmpSmem {
    static constexpr int ROWB = D * 2 + 16;                  // padded row: conflict-free ldmatrix
    static constexpr int STAGE = 2 * CMP_CHUNK * ROWB;       // K then V
    static constexpr int Q_OFF = 2 * STAGE;
    static constexpr int ROPE_OFF = Q_OFF + 16 * ROWB;       // cos/sin of 16 rows x D/2 feature pairs (fused rotary embedding)
    static constexpr int TOTAL = ROPE_OFF + 16 * (D / 2) * 8;
    static constexpr int MERGE_BYTES = CMP_WARPS * 16 * (D + 2) * 4;   // reuses the stages
    static_assert(MERGE_BYTES <= 2 * STAGE, "merge buffer must fit in the stage buffers");
};

template <int D>
__global__ void __launch_bounds__(CMP_WARPS * 32)
compress_mma_kernel(const __nv_bfloat16* __restrict__ q_mem, const __nv_bfloat16* __restrict__ k_mem,
                    const __nv_bfloat16* __restrict__ v_mem, __nv_bfloat16* __restrict__ k_cache,
                    __nv_bfloat16* __restrict__ v_cache, __nv_bfloat16* __restrict__ o_mem, float* __restrict__ lse,
                    float* __restrict__ ws, int BH, int cap, int mem_len_all, const int32_t* __restrict__ mem_lens, int H,
                    int t, int tc, int nprior, int prior_len, int mtiles, float scale_log2, Paging pg, RopeArgs rope) {
    using SM = CmpSmem<D>;
    constexpr int ROWB = SM::ROWB;
    constexpr int VPR = D / 8;                 // 16-byte vectors per row
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(smem);
    // one CTA per (b,h), key range and tile of 16 query rows (t > 16 memory queries take several tiles)
    const int nsp = nprior + 1;
    const int mt = blockIdx.x % mtiles;
    const int bs = blockIdx.x / mtiles;
    const int bh = bs / nsp, split = bs - bh * nsp;
    const bool is_tail = split == nprior;
    // ragged batch (default variant only, nprior == 0): every sequence has its own count of memory entries, clamped
    // to the bound the caller vouched for; a negative count means the sequence does not compress in this call
    int mem_len = mem_len_all;
    if (mem_lens) {
        mem_len = __ldg(mem_lens + bh / H);
        if (mem_len < 0) return;
        mem_len = min(mem_len, mem_len_all);
    }
    const int q0 = mt * 16;                    // first query row of this tile
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;

    // cache slot j of this (b,h) -> element offset from k_cache / v_cache (through the block table when the cache is paged)
    const int pb = bh / H, phd = bh - pb * H;
    auto cache_row = [&](int j) -> int64_t {
        if (!pg.table) return ((int64_t)bh * cap + j) * D;
        const int page = min(max(__ldg(pg.table + (int64_t)pb * pg.max_pages + (j >> pg.log2_ps)), 0), pg.n_pages - 1);
        return ((((int64_t)page * H + phd) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * D;
    };
    const __nv_bfloat16* kc = k_cache;
    const __nv_bfloat16* vc = v_cache;
    const __nv_bfloat16* km = k_mem + (int64_t)bh * t * D;
    const __nv_bfloat16* vm = v_mem + (int64_t)bh * t * D;
    // key i of this CTA's range -> source row
    const int k0 = is_tail ? mem_len : split * prior_len;
    const int n_cache_rows = is_tail ? tc : min(prior_len, mem_len - k0);
    const int nkeys = is_tail ? tc + t : n_cache_rows;

    auto stage_chunk = [&](int ci, int st) {
        const uint32_t kdst = sbase + st * SM::STAGE, vdst = kdst + CMP_CHUNK * ROWB;
        for (int e = threadIdx.x; e < CMP_CHUNK * VPR; e += CMP_WARPS * 32) {
            const int r = e / VPR, cv = e - r * VPR;
            const int i = ci * CMP_CHUNK + r;
            const bool valid = i < nkeys;
            const int ic = valid ? i : 0;
            const __nv_bfloat16 *ksrc, *vsrc;
            if (ic < n_cache_rows) { const int64_t off = cache_row(k0 + ic); ksrc = kc + off; vsrc = vc + off; }
            else { ksrc = km + (int64_t)(ic - n_cache_rows) * D; vsrc = vm + (int64_t)(ic - n_cache_rows) * D; }
            cp_async16(kdst + r * ROWB + cv * 16, ksrc + cv * 8, valid);
            cp_async16(vdst + r * ROWB + cv * 16, vsrc + cv * 8, valid);
        }
    };

    const int nchunks = (nkeys + CMP_CHUNK - 1) / CMP_CHUNK;
    if (nchunks > 0) stage_chunk(0, 0);
    cp_async_commit();

    // queries: 16 rows (rows >= t are zero), staged once, then kept as A fragments
    for (int e = threadIdx.x; e < 16 * VPR; e += CMP_WARPS * 32) {
        const int r = e / VPR, cv = e - r * VPR;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (q0 + r < t) val = __ldg(reinterpret_cast<const uint4*>(q_mem + ((int64_t)bh * t + q0 + r) * D) + cv);
        *reinterpret_cast<uint4*>(smem + SM::Q_OFF + r * ROWB + cv * 16) = val;
    }
    // Fused rotary embedding (Section 4.5): memory row j is rotated by the id pos0 + j * stride -- its query here,
    // its key where it is staged below and where it is written into the cache.  cos/sin per (row, feature pair)
    // are tabulated once per CTA.
    float2* rope_tab = reinterpret_cast<float2*>(smem + SM::ROPE_OFF);
    auto rotate_row_in_smem = [&](uint8_t* row, int j16, int d) {   // features d and d + D/2 of a staged bf16 row
        __nv_bfloat16* x = reinterpret_cast<__nv_bfloat16*>(row);
        const float2 cs = rope_tab[j16 * (D / 2) + d];
        const float a = __bfloat162float(x[d]), b = __bfloat162float(x[d + D / 2]);
        x[d] = __float2bfloat16_rn(a * cs.x - b * cs.y);
        x[d + D / 2] = __float2bfloat16_rn(b * cs.x + a * cs.y);
    };
    if (rope.on) {
        for (int e = threadIdx.x; e < 16 * (D / 2); e += CMP_WARPS * 32) {
            const int r = e / (D / 2), d = e - r * (D / 2);
            float c, sn;
            rope_cos_sin((rope.pos_seq ? __ldg(rope.pos_seq + bh / H) : rope.pos0) + (q0 + r) * rope.stride, d, D, rope.log2_base, c, sn);
            rope_tab[e] = make_float2(c, sn);
        }
        __syncthreads();
        for (int e = threadIdx.x; e < 16 * (D / 2); e += CMP_WARPS * 32) {
            const int r = e / (D / 2), d = e - r * (D / 2);
            if (q0 + r < t) rotate_row_in_smem(smem + SM::Q_OFF + r * ROWB, r, d);
        }
    }
    __syncthreads();
    uint32_t qa[D / 16][4];
    {
        const int mi = lane >> 3;
        const uint32_t row_addr = sbase + SM::Q_OFF + ((mi & 1) * 8 + (lane & 7)) * ROWB + (mi >> 1) * 16;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) ldsm_x4(row_addr + kk * 32, qa[kk]);
    }

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows g and g+8
    float oacc[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; ++j) { oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f; }

    for (int ci = 0; ci < nchunks; ++ci) {
        if (ci + 1 < nchunks) stage_chunk(ci + 1, (ci + 1) & 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        if (rope.on && is_tail && (ci + 1) * CMP_CHUNK > n_cache_rows) {
            // the memory rows' own keys (rows n_cache_rows .. nkeys - 1 of the range) are rotated where they were staged
            uint8_t* kst_gen = smem + (ci & 1) * SM::STAGE;
            for (int e = threadIdx.x; e < CMP_CHUNK * (D / 2); e += CMP_WARPS * 32) {
                const int r = e / (D / 2), d = e - r * (D / 2);
                const int j = ci * CMP_CHUNK + r - n_cache_rows;     // memory row
                if (j >= 0 && j < t) rotate_row_in_smem(kst_gen + r * ROWB, j - q0, d);
            }
            __syncthreads();
        }
        const int kb = ci * CMP_CHUNK + warp * 16;        // this warp's 16 keys
        if (kb < nkeys) {
            const uint32_t kst = sbase + (ci & 1) * SM::STAGE + warp * 16 * ROWB;
            const uint32_t vst = kst + CMP_CHUNK * ROWB;
            float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            {
                const int mi = lane >> 3;
                const uint32_t addr = kst + ((mi >> 1) * 8 + (lane & 7)) * ROWB + (mi & 1) * 16;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    uint32_t kf[4];
                    ldsm_x4(addr + kk * 32, kf);
                    mma_bf16_16816(sc[0], qa[kk], kf[0], kf[1]);
                    mma_bf16_16816(sc[1], qa[kk], kf[2], kf[3]);
                }
            }
            // mask keys beyond the range, then online softmax (exp2 domain)
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool valid = kb + 8 * j + 2 * tq + e < nkeys;
                    sc[j][e] = valid ? sc[j][e] * scale_log2 : -INFINITY;
                    sc[j][2 + e] = valid ? sc[j][2 + e] * scale_log2 : -INFINITY;
                    mx0 = fmaxf(mx0, sc[j][e]);
                    mx1 = fmaxf(mx1, sc[j][2 + e]);
                }
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);   // finite: key kb is valid for every row
            const float a0 = ex2f(m0 - mn0), a1 = ex2f(m1 - mn1);
            m0 = mn0; m1 = mn1;
            uint32_t pa[4];
            {
                const float p00 = ex2f(sc[0][0] - mn0), p01 = ex2f(sc[0][1] - mn0);
                const float p02 = ex2f(sc[0][2] - mn1), p03 = ex2f(sc[0][3] - mn1);
                const float p10 = ex2f(sc[1][0] - mn0), p11 = ex2f(sc[1][1] - mn0);
                const float p12 = ex2f(sc[1][2] - mn1), p13 = ex2f(sc[1][3] - mn1);
                l0 = l0 * a0 + (p00 + p01) + (p10 + p11);
                l1 = l1 * a1 + (p02 + p03) + (p12 + p13);
                pa[0] = pack_bf16(p00, p01);   // (row g,   keys 2t, 2t+1)
                pa[1] = pack_bf16(p02, p03);   // (row g+8, keys 2t, 2t+1)
                pa[2] = pack_bf16(p10, p11);   // (row g,   keys 8+2t, ..)
                pa[3] = pack_bf16(p12, p13);   // (row g+8, keys 8+2t, ..)
            }
#pragma unroll
            for (int j = 0; j < D / 8; ++j) {
                oacc[j][0] *= a0; oacc[j][1] *= a0; oacc[j][2] *= a1; oacc[j][3] *= a1;
            }
            {
                const int mi = lane >> 3;
                const uint32_t addr = vst + ((mi & 1) * 8 + (lane & 7)) * ROWB + (mi >> 1) * 16;
#pragma unroll
                for (int jd = 0; jd < D / 8; jd += 2) {
                    uint32_t vf[4];
                    ldsm_x4_trans(addr + jd * 16, vf);
                    mma_bf16_16816(oacc[jd], pa, vf[0], vf[1]);
                    mma_bf16_16816(oacc[jd + 1], pa, vf[2], vf[3]);
                }
            }
        }
        __syncthreads();   // the stage is refilled two iterations later
    }
    cp_async_wait<0>();
    // row sums live in the four lanes of a quad
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // merge the warps through shared memory (stage buffers are free now)
    float* mg_o = reinterpret_cast<float*>(smem);                          // [warp][16][D]
    float* mg_ml = mg_o + CMP_WARPS * 16 * D;                              // [warp][16][2]
#pragma unroll
    for (int j = 0; j < D / 8; ++j) {
        float* r0 = mg_o + ((warp * 16 + g) * D) + 8 * j + 2 * tq;
        float* r1 = mg_o + ((warp * 16 + g + 8) * D) + 8 * j + 2 * tq;
        r0[0] = oacc[j][0]; r0[1] = oacc[j][1];
        r1[0] = oacc[j][2]; r1[1] = oacc[j][3];
    }
    if (tq == 0) {
        mg_ml[(warp * 16 + g) * 2] = m0; mg_ml[(warp * 16 + g) * 2 + 1] = l0;
        mg_ml[(warp * 16 + g + 8) * 2] = m1; mg_ml[(warp * 16 + g + 8) * 2 + 1] = l1;
    }
    __syncthreads();
    {
        constexpr int SEG = D / 8;               // 8 threads per row, SEG columns each
        const int r = threadIdx.x >> 3, d0 = (threadIdx.x & 7) * SEG;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < CMP_WARPS; ++w) M = fmaxf(M, mg_ml[(w * 16 + r) * 2]);
        float f[CMP_WARPS], lt = 0.f;
#pragma unroll
        for (int w = 0; w < CMP_WARPS; ++w) {
            const float mw = mg_ml[(w * 16 + r) * 2];
            f[w] = (mw > -INFINITY) ? ex2f(mw - M) : 0.f;
            lt = fmaf(mg_ml[(w * 16 + r) * 2 + 1], f[w], lt);
        }
        if (q0 + r < t) {
            if (nsp == 1) {
                const float inv = 1.f / lt;
                __nv_bfloat16* dst = o_mem + ((int64_t)bh * t + q0 + r) * D + d0;
#pragma unroll
                for (int d = 0; d < SEG; d += 2) {
                    float x0 = 0.f, x1 = 0.f;
#pragma unroll
                    for (int w = 0; w < CMP_WARPS; ++w) {
                        x0 = fmaf(mg_o[(w * 16 + r) * D + d0 + d], f[w], x0);
                        x1 = fmaf(mg_o[(w * 16 + r) * D + d0 + d + 1], f[w], x1);
                    }
                    *reinterpret_cast<uint32_t*>(dst + d) = pack_bf16(x0 * inv, x1 * inv);
                }
                if (lse && d0 == 0) lse[(int64_t)bh * t + q0 + r] = (M + log2f(lt)) * 0.6931471805599453f;
            } else {
                const int64_t slot = (((int64_t)bh * nsp + split) * mtiles + mt) * 16 + r;
                float* po = ws + slot * D + d0;
#pragma unroll
                for (int d = 0; d < SEG; ++d) {
                    float x = 0.f;
#pragma unroll
                    for (int w = 0; w < CMP_WARPS; ++w) x = fmaf(mg_o[(w * 16 + r) * D + d0 + d], f[w], x);
                    po[d] = x;
                }
                if (d0 == 0) {
                    float* pml = ws + (int64_t)BH * nsp * mtiles * 16 * D + slot * 2;
                    pml[0] = M; pml[1] = lt;
                }
            }
        }
    }
    // compaction (Section 3.1 step 3): every read of the tail by this launch happened in this CTA, above
    // (with several query tiles per (b,h) other CTAs read the same tail: a separate launch compacts then)
    if (is_tail && mtiles == 1) {
        __syncthreads();
        const uint4* ksrc = reinterpret_cast<const uint4*>(km);
        const uint4* vsrc = reinterpret_cast<const uint4*>(vm);
        for (int e = threadIdx.x; e < t * VPR; e += CMP_WARPS * 32) {
            const int r = e / VPR, cv = e - r * VPR;
            const int64_t off = cache_row(mem_len + r) + cv * 8;
            if (!rope.on) *reinterpret_cast<uint4*>(k_cache + off) = __ldg(ksrc + e);
            *reinterpret_cast<uint4*>(v_cache + off) = __ldg(vsrc + e);
        }
        if (rope.on) {   // the keys go into the cache rotated (the same arithmetic as for the staged copies)
            for (int e = threadIdx.x; e < t * (D / 2); e += CMP_WARPS * 32) {
                const int r = e / (D / 2), d = e - r * (D / 2);
                const float2 cs = rope_tab[r * (D / 2) + d];
                const float a = __bfloat162float(km[(int64_t)r * D + d]), b = __bfloat162float(km[(int64_t)r * D + d + D / 2]);
                const int64_t off = cache_row(mem_len + r);
                k_cache[off + d] = __float2bfloat16_rn(a * cs.x - b * cs.y);
                k_cache[off + d + D / 2] = __float2bfloat16_rn(b * cs.x + a * cs.y);
            }
        }
    }
}

// ------------------------------------------------------------------ default mask, short ranges: the range in one stage
// Default mask and t <= 16: the key range of a (b,h) is the tc tail rows plus the t memory rows' own keys
// (80 keys for c = 4, t = 16).  A range that short fits one stage: the CTA (one per (b,h)) issues every load
// at once and walks no pipeline.  The warps split the scores by key (8 keys per tensor-core tile), the softmax
// runs over full rows held in shared memory (8 threads per row), and each warp then owns D/4 output columns
// over all keys: nothing is merged across warps.  The compaction writes the staged (with the fused rotary
// embedding: rotated) copies of the memory rows, so k_mem / v_mem are read once.  56 KB of shared memory at
// 80 keys: four CTAs (16 warps) per SM.  (A persistent CTA that loads the next (b,h) while it computes the
// current one was measured slower: its two buffers leave two CTAs per SM, too few warps to cover the
// latencies of the arithmetic.)
struct CmpOneStageLayout {
    int rowb;       // K / V / Q row in bytes, unpadded: 16-byte chunk c of row r lies at chunk c ^ (r & 7), which keeps
                    // ldmatrix free of bank conflicts without the padding (five CTAs per SM at 80 keys instead of four)
    int srow;       // fp32 scores per row
    int prowb;      // bf16 probabilities per row, padded
    int kv_bytes;   // K rows, V rows, Q rows
    int s_off, p_off, ml_off, rope_off, total;   // scores and probabilities lie over the K rows, which are dead by then
};
__host__ __device__ inline CmpOneStageLayout cmp_one_stage_layout(int D, int nk16, bool rope) {
    CmpOneStageLayout l;
    l.rowb = D * 2;
    l.srow = nk16 + 4;
    l.prowb = nk16 * 2 + 16;
    l.kv_bytes = (2 * nk16 + 16) * l.rowb;
    l.s_off = 0;                               // 16 * (nk16 + 4) * 4 + 16 * (2 nk16 + 16) <= nk16 * rowb for nk16 >= 16
    l.p_off = l.s_off + 16 * l.srow * 4;
    l.ml_off = l.kv_bytes;
    l.rope_off = l.ml_off + 32 * 4;
    l.total = l.rope_off + (rope ? 16 * (D / 2) * 8 : 0);
    return l;
}
constexpr int CMP_ONE_STAGE_MAX_SMEM = 72 * 1024;       // three CTAs of four warps per SM (nk16 <= 96: three 8-key tiles a warp)
constexpr int CMP_ONE_STAGE_MAX_SMEM_8W = 110 * 1024;   // two CTAs of eight warps per SM; longer ranges take the pipelined kernel

template <int D, int WARPS>
__global__ void __launch_bounds__(WARPS * 32)
compress_one_stage_kernel(const __nv_bfloat16* __restrict__ q_mem, const __nv_bfloat16* __restrict__ k_mem,
                      const __nv_bfloat16* __restrict__ v_mem, __nv_bfloat16* __restrict__ k_cache,
                      __nv_bfloat16* __restrict__ v_cache, __nv_bfloat16* __restrict__ o_mem, float* __restrict__ lse,
                      int cap, int mem_len_all, const int32_t* __restrict__ mem_lens, int H, int t, int tc,
                      float scale_log2, Paging pg, RopeArgs rope) {
    constexpr int VPR = D / 8;                 // 16-byte vectors per row
    constexpr int NTH = WARPS * 32;
    constexpr int TPR = NTH / 16;              // threads per row in the softmax
    static_assert(D % (8 * WARPS) == 0 && (D / (8 * WARPS)) % 2 == 0, "a warp owns an even number of 8-column tiles");
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(smem);
    const int nkeys = tc + t;
    const int nk16 = (nkeys + 15) & ~15;           // rows past nkeys are zero: their probabilities are zero too
    const CmpOneStageLayout lay = cmp_one_stage_layout(D, nk16, rope.on != 0);
    const int ROWB = lay.rowb;
    const int K_OFF = 0, V_OFF = nk16 * ROWB, Q_OFF = 2 * nk16 * ROWB;
    auto sw = [&](int row, int chunk) -> int { return row * ROWB + ((chunk ^ (row & 7)) << 4); };   // byte offset of a 16-byte chunk
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3, mi = lane >> 3;

    // ragged batch: every sequence has its own count of memory entries, clamped to the bound the caller vouched
    // for; a negative count means the sequence does not compress in this call
    auto own_mem_len = [&](int bh) -> int {
        if (!mem_lens) return mem_len_all;
        const int m = __ldg(mem_lens + bh / H);
        return m < 0 ? -1 : min(m, mem_len_all);
    };
    // cache slot j of (b,h) -> element offset from k_cache / v_cache (through the block table when the cache is paged)
    auto cache_row = [&](int bh, int j) -> int64_t {
        if (!pg.table) return ((int64_t)bh * cap + j) * D;
        const int pb = bh / H, phd = bh - pb * H;
        const int page = min(max(__ldg(pg.table + (int64_t)pb * pg.max_pages + (j >> pg.log2_ps)), 0), pg.n_pages - 1);
        return ((((int64_t)page * H + phd) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * D;
    };
    const int bh = blockIdx.x;
    const int mem_len = own_mem_len(bh);
    if (mem_len < 0) return;
    // every load at once: the tail rows of the cache, the memory rows' own keys and values, the queries
    const uint32_t base = sbase;
    const __nv_bfloat16* km = k_mem + (int64_t)bh * t * D;
    const __nv_bfloat16* vm = v_mem + (int64_t)bh * t * D;
    for (int e = threadIdx.x; e < nk16 * VPR; e += NTH) {
        const int r = e / VPR, cv = e - r * VPR;
        const bool valid = r < nkeys;
        const __nv_bfloat16 *ksrc = km, *vsrc = vm;
        if (valid) {
            if (r < tc) { const int64_t off = cache_row(bh, mem_len + r); ksrc = k_cache + off; vsrc = v_cache + off; }
            else { ksrc = km + (int64_t)(r - tc) * D; vsrc = vm + (int64_t)(r - tc) * D; }
        }
        cp_async16(base + K_OFF + sw(r, cv), ksrc + cv * 8, valid);
        cp_async16(base + V_OFF + sw(r, cv), vsrc + cv * 8, valid);
    }
    for (int e = threadIdx.x; e < 16 * VPR; e += NTH) {
        const int r = e / VPR, cv = e - r * VPR;
        const bool valid = r < t;          // query rows >= t are zero
        cp_async16(base + Q_OFF + sw(r, cv), q_mem + ((int64_t)bh * t + (valid ? r : 0)) * D + cv * 8, valid);
    }
    cp_async_commit();

    float* S = reinterpret_cast<float*>(smem + lay.s_off);
    float* ml = reinterpret_cast<float*>(smem + lay.ml_off);
    float2* rope_tab = reinterpret_cast<float2*>(smem + lay.rope_off);

    // Fused rotary embedding (Section 4.5), as in compress_mma_kernel: memory row j turns by the id
    // pos0 + j * stride; the table is computed while the loads are in flight.
    if (rope.on) {
        const int pos0 = rope.pos_seq ? __ldg(rope.pos_seq + bh / H) : rope.pos0;
        for (int e = threadIdx.x; e < t * (D / 2); e += NTH) {
            const int r = e / (D / 2), d = e - r * (D / 2);
            float c, sn;
            rope_cos_sin(pos0 + r * rope.stride, d, D, rope.log2_base, c, sn);
            rope_tab[e] = make_float2(c, sn);
        }
    }
    cp_async_wait<0>();
    __syncthreads();
    if (rope.on) {
        // the queries and the staged copies of the memory rows' own keys, each pair of features once
        for (int e = threadIdx.x; e < 2 * t * (D / 2); e += NTH) {
            const int which = e / (t * (D / 2)), e2 = e - which * t * (D / 2);
            const int r = e2 / (D / 2), d = e2 - r * (D / 2);
            const int row = which ? tc + r : r;
            uint8_t* rowp = smem + (which ? K_OFF : Q_OFF);
            __nv_bfloat16* xa = reinterpret_cast<__nv_bfloat16*>(rowp + sw(row, d >> 3)) + (d & 7);
            __nv_bfloat16* xb = reinterpret_cast<__nv_bfloat16*>(rowp + sw(row, (d + D / 2) >> 3)) + (d & 7);
            const float2 cs = rope_tab[r * (D / 2) + d];
            const float a = __bfloat162float(*xa), b = __bfloat162float(*xb);
            *xa = __float2bfloat16_rn(a * cs.x - b * cs.y);
            *xb = __float2bfloat16_rn(b * cs.x + a * cs.y);
        }
        __syncthreads();
    }
    // Compaction (Section 3.1 step 3): this CTA is the only reader of cache slots [mem_len, mem_len + t) of
    // this (b,h) in the launch and its copies of them have landed; the slots now take the staged memory rows.
    for (int e = threadIdx.x; e < t * VPR; e += NTH) {
        const int r = e / VPR, cv = e - r * VPR;
        const int64_t off = cache_row(bh, mem_len + r) + cv * 8;
        *reinterpret_cast<uint4*>(k_cache + off) = *reinterpret_cast<const uint4*>(smem + K_OFF + sw(tc + r, cv));
        *reinterpret_cast<uint4*>(v_cache + off) = *reinterpret_cast<const uint4*>(smem + V_OFF + sw(tc + r, cv));
    }

    // scores: tensor-core tiles of 8 keys, dealt to the warps round robin
    {
        constexpr int MAXT = 3;                    // 8-key tiles per warp (the launcher keeps nk16 / 8 <= MAXT * WARPS)
        uint32_t qa[D / 16][4];
        const int qr = (mi & 1) * 8 + (lane & 7);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) ldsm_x4(base + Q_OFF + sw(qr, 2 * kk + (mi >> 1)), qa[kk]);
        float sc[MAXT][4];
#pragma unroll
        for (int i = 0; i < MAXT; ++i) {
            sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
            const int nt = warp + i * WARPS;
            if (nt < nk16 / 8) {
                const int kr = nt * 8 + (lane & 7);
#pragma unroll
                for (int k2 = 0; k2 < D / 32; ++k2) {
                    uint32_t kf[4];   // 8 keys x 32 features: the B fragments of two k-steps
                    ldsm_x4(base + K_OFF + sw(kr, 4 * k2 + mi), kf);
                    mma_bf16_16816(sc[i], qa[2 * k2], kf[0], kf[1]);
                    mma_bf16_16816(sc[i], qa[2 * k2 + 1], kf[2], kf[3]);
                }
            }
        }
        __syncthreads();   // every read of the K rows (score products, compaction) is done: the scores go over them
#pragma unroll
        for (int i = 0; i < MAXT; ++i) {
            const int nt = warp + i * WARPS;
            if (nt < nk16 / 8) {
                const int col = nt * 8 + 2 * tq;
                const bool v0 = col < nkeys, v1 = col + 1 < nkeys;
                *reinterpret_cast<float2*>(S + g * lay.srow + col) =
                    make_float2(v0 ? sc[i][0] * scale_log2 : -INFINITY, v1 ? sc[i][1] * scale_log2 : -INFINITY);
                *reinterpret_cast<float2*>(S + (g + 8) * lay.srow + col) =
                    make_float2(v0 ? sc[i][2] * scale_log2 : -INFINITY, v1 ? sc[i][3] * scale_log2 : -INFINITY);
            }
        }
    }
    __syncthreads();
    // softmax over full rows (exp2 domain): TPR threads per row, two passes over the row in shared memory;
    // key 0 is valid for every row, so the maximum is finite
    {
        const int r = threadIdx.x / TPR, sub = threadIdx.x % TPR;
        const float* srow = S + r * lay.srow;
        __nv_bfloat16* prow = reinterpret_cast<__nv_bfloat16*>(smem + lay.p_off + r * lay.prowb);
        float mx = -INFINITY;
        for (int j = sub; j < nk16; j += TPR) mx = fmaxf(mx, srow[j]);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
        if (TPR == 16) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        float sum = 0.f;
        for (int j = sub; j < nk16; j += TPR) {
            const float pr = ex2f(srow[j] - mx);
            sum += pr;
            prow[j] = __float2bfloat16_rn(pr);
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        sum += __shfl_xor_sync(0xffffffffu, sum, 4);
        if (TPR == 16) sum += __shfl_xor_sync(0xffffffffu, sum, 8);
        if (sub == 0) { ml[r] = mx; ml[16 + r] = sum; }
    }
    __syncthreads();
    // O = P V: each warp owns D / WARPS output columns over every key
    {
        constexpr int NT = D / (8 * WARPS);     // 8-column tiles per warp
        float oacc[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) { oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f; }
        const uint32_t prow = sbase + lay.p_off + ((mi & 1) * 8 + (lane & 7)) * lay.prowb + (mi >> 1) * 16;
        const int vr = (mi & 1) * 8 + (lane & 7), vchunk = (mi >> 1) + warp * (D / WARPS) / 8;
        for (int ks = 0; ks < nk16 / 16; ++ks) {
            uint32_t pa[4];
            ldsm_x4(prow + ks * 32, pa);
#pragma unroll
            for (int jd = 0; jd < NT; jd += 2) {
                uint32_t vf[4];
                ldsm_x4_trans(base + V_OFF + sw(ks * 16 + vr, vchunk + jd), vf);
                mma_bf16_16816(oacc[jd], pa, vf[0], vf[1]);
                mma_bf16_16816(oacc[jd + 1], pa, vf[2], vf[3]);
            }
        }
        const float inv0 = 1.f / ml[16 + g], inv1 = 1.f / ml[16 + g + 8];
        __nv_bfloat16* o0 = o_mem + ((int64_t)bh * t + g) * D + warp * (D / WARPS) + 2 * tq;
        __nv_bfloat16* o1 = o0 + 8 * D;
#pragma unroll
        for (int jd = 0; jd < NT; ++jd) {
            if (g < t) *reinterpret_cast<uint32_t*>(o0 + jd * 8) = pack_bf16(oacc[jd][0] * inv0, oacc[jd][1] * inv0);
            if (g + 8 < t) *reinterpret_cast<uint32_t*>(o1 + jd * 8) = pack_bf16(oacc[jd][2] * inv1, oacc[jd][3] * inv1);
        }
    }
    if (lse && threadIdx.x < t)
        lse[(int64_t)bh * t + threadIdx.x] = (ml[threadIdx.x] + log2f(ml[16 + threadIdx.x])) * 0.6931471805599453f;
}

template <int D>
__global__ void __launch_bounds__(D)
compress_merge_kernel(const float* __restrict__ ws, __nv_bfloat16* __restrict__ o_mem, float* __restrict__ lse,
                      int BH, int t, int nsp, int mtiles) {
    const int bh = blockIdx.x / t, r = blockIdx.x - bh * t, d = threadIdx.x;
    const int mt = r >> 4, r16 = r & 15;
    const float* pml = ws + (int64_t)BH * nsp * mtiles * 16 * D;
    auto slot = [&](int s) { return (((int64_t)bh * nsp + s) * mtiles + mt) * 16 + r16; };
    float M = -INFINITY;
    for (int s = 0; s < nsp; ++s) M = fmaxf(M, pml[slot(s) * 2]);
    float lt = 0.f, ot = 0.f;
    for (int s = 0; s < nsp; ++s) {
        const float ms = pml[slot(s) * 2];
        if (ms > -INFINITY) {
            const float f = exp2f(ms - M);
            lt = fmaf(pml[slot(s) * 2 + 1], f, lt);
            ot = fmaf(ws[slot(s) * D + d], f, ot);
        }
    }
    o_mem[((int64_t)bh * t + r) * D + d] = __float2bfloat16_rn(ot / lt);
    if (lse && d == 0) lse[(int64_t)bh * t + r] = (M + log2f(lt)) * 0.6931471805599453f;
}

// Compaction on its own (used when the memory queries span several 16-row tiles): runs after the
// attention kernel in stream order, so every read of the tail has completed.
template <int D>
__global__ void compaction_kernel(const __nv_bfloat16* __restrict__ k_mem, const __nv_bfloat16* __restrict__ v_mem,
                                  __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache, int cap,
                                  int mem_len, const int32_t* __restrict__ mem_lens, int H, int t, Paging pg) {
    const int bh = blockIdx.x;
    if (mem_lens) {
        const int own = __ldg(mem_lens + bh / H);
        if (own < 0) return;
        mem_len = min(own, mem_len);
    }
    constexpr int VPR = D / 8;
    const uint4* ksrc = reinterpret_cast<const uint4*>(k_mem + (int64_t)bh * t * D);
    const uint4* vsrc = reinterpret_cast<const uint4*>(v_mem + (int64_t)bh * t * D);
    const int pb = bh / H, phd = bh - pb * H;
    for (int e = threadIdx.x; e < t * VPR; e += blockDim.x) {
        const int r = e / VPR, cv = e - r * VPR, j = mem_len + r;
        int64_t off;
        if (!pg.table) {
            off = ((int64_t)bh * cap + j) * D;
        } else {
            const int page = min(max(__ldg(pg.table + (int64_t)pb * pg.max_pages + (j >> pg.log2_ps)), 0), pg.n_pages - 1);
            off = ((((int64_t)page * H + phd) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * D;
        }
        *reinterpret_cast<uint4*>(k_cache + off + cv * 8) = __ldg(ksrc + e);
        *reinterpret_cast<uint4*>(v_cache + off + cv * 8) = __ldg(vsrc + e);
    }
}

template <int D>
static cudaError_t compress_bf16_t(const void* qm, const void* km, const void* vm, void* kc, void* vc, void* om,
                                   float* lse, int BH, int cap, int mem_len, const int32_t* mem_lens, int H, int t, int tc,
                                   unsigned flags, float scale, void* ws, const Paging& pg, cudaStream_t st,
                                   const RopeArgs& rope) {
    const int nprior = compress_num_prior(BH, mem_len, flags);
    int prior_len = 0;
    if (nprior > 0) prior_len = ((mem_len + nprior - 1) / nprior + 15) / 16 * 16;
    const int nsp = nprior + 1;
    const int nk16 = (tc + t + 15) & ~15;
    const CmpOneStageLayout wl = cmp_one_stage_layout(D, nk16, rope.on != 0);
    // default mask, short range: the whole range in one stage.  A warp holds the scores of at most three 8-key tiles:
    // four warps up to 96 keys, eight (D = 128 only: a warp owns at least 16 output columns) up to 192, and two CTAs an SM
    const bool narrow = nk16 <= 96 && wl.total <= CMP_ONE_STAGE_MAX_SMEM;
    const bool wide8 = !narrow && D == 128 && nk16 <= 192 && wl.total <= CMP_ONE_STAGE_MAX_SMEM_8W;
    if (nprior == 0 && t <= 16 && (narrow || wide8)) {
        constexpr int W8 = D == 128 ? 8 : 4;
        const bool wide = wide8;
        static bool attr1_set[64] = {false};   // per device, per template instance
        int dev1 = 0;
        if (cudaGetDevice(&dev1) != cudaSuccess || dev1 < 0 || dev1 >= 64) return cudaErrorInvalidDevice;
        if (!attr1_set[dev1]) {
            cudaError_t e1 = cudaFuncSetAttribute(compress_one_stage_kernel<D, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  CMP_ONE_STAGE_MAX_SMEM);
            if (e1 == cudaSuccess)
                e1 = cudaFuncSetAttribute(compress_one_stage_kernel<D, W8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          CMP_ONE_STAGE_MAX_SMEM_8W);
            if (e1 != cudaSuccess) return e1;
            attr1_set[dev1] = true;
        }
        auto kern = wide ? compress_one_stage_kernel<D, W8> : compress_one_stage_kernel<D, 4>;
        kern<<<BH, (wide ? W8 : 4) * 32, wl.total, st>>>(
            static_cast<const __nv_bfloat16*>(qm), static_cast<const __nv_bfloat16*>(km),
            static_cast<const __nv_bfloat16*>(vm), static_cast<__nv_bfloat16*>(kc), static_cast<__nv_bfloat16*>(vc),
            static_cast<__nv_bfloat16*>(om), lse, cap, mem_len, mem_lens, H, t, tc, scale * 1.4426950408889634f, pg, rope);
        count_launches(1);
        return cudaGetLastError();
    }
    // (the cos/sin table of the fused rotary embedding is only allocated when it is used: without it three CTAs fit an SM)
    const int smem = rope.on ? CmpSmem<D>::TOTAL : CmpSmem<D>::ROPE_OFF;
    cudaError_t e;
    static bool attr_set[64] = {false};   // per device, per template instance
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(compress_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, CmpSmem<D>::TOTAL);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int mtiles = (t + 15) / 16;
    compress_mma_kernel<D><<<BH * nsp * mtiles, CMP_WARPS * 32, smem, st>>>(
        static_cast<const __nv_bfloat16*>(qm), static_cast<const __nv_bfloat16*>(km),
        static_cast<const __nv_bfloat16*>(vm), static_cast<__nv_bfloat16*>(kc), static_cast<__nv_bfloat16*>(vc),
        static_cast<__nv_bfloat16*>(om), lse, static_cast<float*>(ws), BH, cap, mem_len, mem_lens, H, t, tc, nprior,
        prior_len, mtiles, scale * 1.4426950408889634f, pg, rope);
    count_launches(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (nsp > 1) {
        compress_merge_kernel<D><<<BH * t, D, 0, st>>>(static_cast<const float*>(ws), static_cast<__nv_bfloat16*>(om),
                                                       lse, BH, t, nsp, mtiles);
        count_launches(1);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (mtiles > 1) {
        compaction_kernel<D><<<BH, 128, 0, st>>>(static_cast<const __nv_bfloat16*>(km),
                                                  static_cast<const __nv_bfloat16*>(vm), static_cast<__nv_bfloat16*>(kc),
                                                  static_cast<__nv_bfloat16*>(vc), cap, mem_len, mem_lens, H, t, pg);
        count_launches(1);
        e = cudaGetLastError();
    }
    return e;
}

// t <= 128 (with the fused rotary embedding: t <= 16); the caller falls back to the CUDA-core kernel otherwise.
cudaError_t launch_compress_bf16(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache, void* v_cache,
                                 void* o_mem, float* lse, int B, int H, int D, int cap, int mem_len,
                                 const int32_t* mem_lens, int c, int t, unsigned flags, float scale, void* ws,
                                 const Paging& pg, cudaStream_t st, const RopeArgs& rope) {
    const int BH = B * H, tc = c * t;
    if (rope.on && t > 16) return cudaErrorNotSupported;
    return D == 64 ? compress_bf16_t<64>(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, BH, cap, mem_len, mem_lens, H, t,
                                         tc, flags, scale, ws, pg, st, rope)
                   : compress_bf16_t<128>(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, BH, cap, mem_len, mem_lens, H, t,
                                          tc, flags, scale, ws, pg, st, rope);
}

}  // namespace loma
