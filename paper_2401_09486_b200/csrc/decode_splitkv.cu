// Split-KV decode attention over the compressed cache (bf16, fp32 accumulate).
//
// One query per (batch, head) attends to cache[0, len) and to itself
// (Appendix A, inference_input with one token).  With one query row there is
// nothing to reuse: every K and V byte is read once, so the kernel is bound by
// HBM bandwidth and is written as a streaming reduction on the CUDA cores.
//
//   grid  = B*H*splits CTAs; each owns a contiguous key range of one (b,h)
//   warp  = takes blocks of 8 row-loads from that range, round robin
//   lanes = LPK = D/8 lanes share one K (or V) row, 16 bytes each, so a warp
//           load instruction covers 32/LPK whole rows, fully coalesced
//   softmax = online, in the exp2 domain; row maxima and sums are combined with
//           warp shuffles, then across the CTA's warps in shared memory
//   merge = partial (m, l, o) of every split go to the workspace and a second
//           small kernel combines them in a fixed order (bitwise repeatable)
#include <math.h>

#include "loma_internal.cuh"

namespace loma {

constexpr int DEC_WARPS = 4;
constexpr int DEC_NL = 8;            // row-loads in flight per lane for K, and again for V
constexpr int DEC_MIN_SPLIT = 256;   // never cut a (b,h) into ranges shorter than this
constexpr int DEC_MAX_SPLITS = 128;

// Number of key ranges a (b,h) is cut into.  Depends only on the arguments, so
// results are repeatable and the workspace size can be computed up front.
int decode_num_splits(int BH, int total_keys) {
    int by_len = (total_keys + 1023) / 1024;               // ~1024 keys per CTA when there are many (b,h)
    int by_fill = (4 * 148 + BH - 1) / BH;                 // enough CTAs for every SM when there are few
    int splits = by_len > by_fill ? by_len : by_fill;
    int cap = total_keys / DEC_MIN_SPLIT;
    if (splits > cap) splits = cap;
    if (splits > DEC_MAX_SPLITS) splits = DEC_MAX_SPLITS;
    if (splits < 1) splits = 1;
    return splits;
}

size_t decode_workspace_bytes(int BH, int D, int total_keys) {
    const int splits = decode_num_splits(BH, total_keys);
    if (splits == 1) return 0;
    return (size_t)BH * splits * (D + 2) * sizeof(float);
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ float dot8(const float (&q)[8], const uint4& k) {
    float a = q[0] * bf16lo(k.x);
    float b = q[1] * bf16hi(k.x);
    a = fmaf(q[2], bf16lo(k.y), a);
    b = fmaf(q[3], bf16hi(k.y), b);
    a = fmaf(q[4], bf16lo(k.z), a);
    b = fmaf(q[5], bf16hi(k.z), b);
    a = fmaf(q[6], bf16lo(k.w), a);
    b = fmaf(q[7], bf16hi(k.w), b);
    return a + b;
}

__device__ __forceinline__ void axpy8(float (&o)[8], float p, const uint4& v) {
    o[0] = fmaf(p, bf16lo(v.x), o[0]);
    o[1] = fmaf(p, bf16hi(v.x), o[1]);
    o[2] = fmaf(p, bf16lo(v.y), o[2]);
    o[3] = fmaf(p, bf16hi(v.y), o[3]);
    o[4] = fmaf(p, bf16lo(v.z), o[4]);
    o[5] = fmaf(p, bf16hi(v.z), o[5]);
    o[6] = fmaf(p, bf16lo(v.w), o[6]);
    o[7] = fmaf(p, bf16hi(v.w), o[7]);
}

// total = cache_len + 1 visible keys; key index cache_len is the new token.
// PAGED: the cache is a pool of pages [n_pages, H, page_size, D]; slot j of sequence b lives in page
// table[b][j / page_size] at row j % page_size (page numbers are clamped to the pool on the device).
template <int D, bool PAGED>
__global__ void __launch_bounds__(DEC_WARPS * 32)
decode_splitkv_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_new,
                      const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ k_cache,
                      __nv_bfloat16* __restrict__ v_cache, __nv_bfloat16* __restrict__ o,
                      float* __restrict__ lse, float* __restrict__ ws, int BH, int cap, int cache_len_max,
                      const int32_t* __restrict__ lens, int H, int splits, int split_len, float scale_log2, Paging pg,
                      RopeArgs rope) {
    constexpr int LPK = D / 8;           // lanes per row
    constexpr int KPL = 32 / LPK;        // rows per warp load
    constexpr int BK = DEC_NL * KPL;     // rows per warp iteration
    __shared__ float sm_m[DEC_WARPS], sm_l[DEC_WARPS];
    __shared__ __align__(16) float sm_o[DEC_WARPS][D];
    // fused rotary embedding (Section 4.5): cos/sin of the step's position per feature pair, and the rotated new key
    __shared__ float sm_cs[D / 2], sm_sn[D / 2];
    __shared__ __align__(16) __nv_bfloat16 sm_kn[D];

    const int bh = blockIdx.x / splits, split = blockIdx.x - bh * splits;
    // ragged batch: every sequence has its own length (clamped to the bound the launch was sized for);
    // ranges beyond a sequence's end are empty and contribute nothing to the merge
    const int cache_len = lens ? min(max(__ldg(lens + bh / H), 0), cache_len_max) : cache_len_max;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / LPK;          // which of the KPL rows of a load this lane works on
    const int li = lane % LPK;           // 16-byte column of the row
    const int total = cache_len + 1;
    const int k_begin = split * split_len;
    const int k_end = min(total, k_begin + split_len);   // may be <= k_begin in a ragged batch

    // slot j of this (b,h) -> offset of its row in 16-byte units from kc / vc
    const int pb = bh / H, phd = bh - pb * H;
    auto row_off = [&](int j) -> int64_t {
        if (!PAGED) return (int64_t)j * LPK;
        const int page = min(max(__ldg(pg.table + (int64_t)pb * pg.max_pages + (j >> pg.log2_ps)), 0), pg.n_pages - 1);
        return ((((int64_t)page * H + phd) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * LPK;
    };
    const uint4* kc = reinterpret_cast<const uint4*>(PAGED ? k_cache : k_cache + (int64_t)bh * cap * D);
    const uint4* vc = reinterpret_cast<const uint4*>(PAGED ? v_cache : v_cache + (int64_t)bh * cap * D);
    const int64_t new_off = row_off(cache_len);
    const uint4* kn = k_new ? reinterpret_cast<const uint4*>(k_new + (int64_t)bh * D) : kc + new_off;
    const uint4* vn = v_new ? reinterpret_cast<const uint4*>(v_new + (int64_t)bh * D) : vc + new_off;

    float qf[8];
    {
        const uint4 qv = __ldg(reinterpret_cast<const uint4*>(q + (int64_t)bh * D) + li);
        qf[0] = bf16lo(qv.x); qf[1] = bf16hi(qv.x); qf[2] = bf16lo(qv.y); qf[3] = bf16hi(qv.y);
        qf[4] = bf16lo(qv.z); qf[5] = bf16hi(qv.z); qf[6] = bf16lo(qv.w); qf[7] = bf16hi(qv.w);
    }
    // does this CTA read the new key (index cache_len) or write it to the cache?
    const bool needs_new_key = (k_begin <= cache_len && cache_len < k_end) || split == splits - 1;
    if (rope.on) {
        // q and the new key are rotated here, in registers / shared memory, by the step's position id: no
        // separate pass over them.  The rotated key, rounded to bf16, is what the step attends to and appends.
        const int pos = rope.pos_seq ? __ldg(rope.pos_seq + bh / H) : rope.pos0;
        if (threadIdx.x < D / 2) rope_cos_sin(pos, threadIdx.x, D, rope.log2_base, sm_cs[threadIdx.x], sm_sn[threadIdx.x]);
        __syncthreads();
        if (needs_new_key && threadIdx.x < D / 2) {
            const __nv_bfloat16* kp = reinterpret_cast<const __nv_bfloat16*>(kn);
            const float a = __bfloat162float(kp[threadIdx.x]), b = __bfloat162float(kp[threadIdx.x + D / 2]);
            const float c = sm_cs[threadIdx.x], sn = sm_sn[threadIdx.x];
            sm_kn[threadIdx.x] = __float2bfloat16_rn(a * c - b * sn);
            sm_kn[threadIdx.x + D / 2] = __float2bfloat16_rn(b * c + a * sn);
        }
        const bool second = li >= LPK / 2;                 // this lane holds features of the second half
        const int dh = (li % (LPK / 2)) * 8;               // its first feature pair
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float other = __shfl_xor_sync(0xffffffffu, qf[e], LPK / 2);
            const float c = sm_cs[dh + e], sn = sm_sn[dh + e];
            qf[e] = second ? qf[e] * c + other * sn : qf[e] * c - other * sn;
        }
        __syncthreads();                                   // sm_kn is read below
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) qf[e] *= scale_log2;

    float m = -INFINITY, l = 0.f;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;

    // Paged cache: a row's address hangs on a block-table entry.  The entries of the next iteration's rows are
    // fetched while this iteration's rows stream in, so no data load waits for a table load issued just before it.
    int64_t off_cur[DEC_NL], off_nxt[DEC_NL];
    auto row_offs = [&](int j0, int64_t* o) {
#pragma unroll
        for (int i = 0; i < DEC_NL; ++i) o[i] = row_off(min(min(j0 + i * KPL + sub, cache_len), max(cache_len - 1, 0)));
    };
    if (PAGED) row_offs(k_begin + warp * BK, off_cur);
    for (int j0 = k_begin + warp * BK; j0 < k_end; j0 += DEC_WARPS * BK) {
        uint4 kr[DEC_NL], vr[DEC_NL];
        bool valid[DEC_NL];
        if (PAGED) row_offs(j0 + DEC_WARPS * BK, off_nxt);
#pragma unroll
        for (int i = 0; i < DEC_NL; ++i) {
            const int j = j0 + i * KPL + sub;
            valid[i] = j < k_end;
            const int jc = min(j, cache_len);                  // stay inside [0, cache_len]
            const uint4* kp = (jc < cache_len) ? kc + (PAGED ? off_cur[i] : row_off(jc)) : kn;
            if (rope.on && jc >= cache_len) kr[i] = *(reinterpret_cast<const uint4*>(sm_kn) + li);   // the rotated new key
            else kr[i] = ld_stream(kp + li);
        }
#pragma unroll
        for (int i = 0; i < DEC_NL; ++i) {
            const int jc = min(j0 + i * KPL + sub, cache_len);
            const uint4* vp = (jc < cache_len) ? vc + (PAGED ? off_cur[i] : row_off(jc)) : vn;
            vr[i] = ld_stream(vp + li);
        }
        if (PAGED) {
#pragma unroll
            for (int i = 0; i < DEC_NL; ++i) off_cur[i] = off_nxt[i];
        }
        float s[DEC_NL];
#pragma unroll
        for (int i = 0; i < DEC_NL; ++i) s[i] = dot8(qf, kr[i]);
#pragma unroll
        for (int off = LPK / 2; off > 0; off >>= 1) {
#pragma unroll
            for (int i = 0; i < DEC_NL; ++i) s[i] += __shfl_xor_sync(0xffffffffu, s[i], off);
        }
        float mb = -INFINITY;
#pragma unroll
        for (int i = 0; i < DEC_NL; ++i) {
            s[i] = valid[i] ? s[i] : -INFINITY;
            mb = fmaxf(mb, s[i]);
        }
#pragma unroll
        for (int off = 16; off >= LPK; off >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, off));
        const float m_new = fmaxf(m, mb);      // finite: the block has at least one valid row
        const float alpha = exp2f(m - m_new);
        l *= alpha;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] *= alpha;
#pragma unroll
        for (int i = 0; i < DEC_NL; ++i) {
            const float p = exp2f(s[i] - m_new);
            l += p;
            axpy8(acc, p, vr[i]);
        }
        m = m_new;
    }
    // rows of one load sit in different lane groups: add the groups up
#pragma unroll
    for (int off = 16; off >= LPK; off >>= 1) {
        l += __shfl_xor_sync(0xffffffffu, l, off);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], off);
    }
    if (lane < LPK) {
        float4* dst = reinterpret_cast<float4*>(&sm_o[warp][lane * 8]);
        dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    }
    if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
    __syncthreads();

    // combine the warps (fixed order), then write the split's partial or the final row
    if (threadIdx.x < D) {
        const int d = threadIdx.x;
        float M = sm_m[0];
#pragma unroll
        for (int w = 1; w < DEC_WARPS; ++w) M = fmaxf(M, sm_m[w]);
        float lt = 0.f, ot = 0.f;
        if (M > -INFINITY) {
#pragma unroll
            for (int w = 0; w < DEC_WARPS; ++w) {
                const float f = exp2f(sm_m[w] - M);
                lt = fmaf(sm_l[w], f, lt);
                ot = fmaf(sm_o[w][d], f, ot);
            }
        }
        if (splits == 1) {
            o[(int64_t)bh * D + d] = __float2bfloat16_rn(ot / lt);
            if (lse && d == 0) lse[bh] = (M + log2f(lt)) * 0.6931471805599453f;
        } else {
            float* po = ws + ((int64_t)bh * splits + split) * D;
            float* pml = ws + (int64_t)BH * splits * D + ((int64_t)bh * splits + split) * 2;
            po[d] = ot;
            if (d == 0) { pml[0] = M; pml[1] = lt; }
        }
    }
    // append the new token's K/V at slot cache_len (read by nobody in this launch)
    if (k_new && split == splits - 1 && warp == 0 && lane < LPK) {
        uint4* kd = const_cast<uint4*>(kc) + new_off;
        uint4* vd = const_cast<uint4*>(vc) + new_off;
        kd[lane] = rope.on ? *(reinterpret_cast<const uint4*>(sm_kn) + lane) : __ldg(kn + lane);
        vd[lane] = __ldg(vn + lane);
    }
}

template <int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const float* __restrict__ ws, __nv_bfloat16* __restrict__ o, float* __restrict__ lse,
                    int splits) {
    const int bh = blockIdx.x, d = threadIdx.x;
    const float* po = ws + (int64_t)bh * splits * D;
    const float* pml = ws + (int64_t)gridDim.x * splits * D + (int64_t)bh * splits * 2;
    float M = -INFINITY;
    for (int s = 0; s < splits; ++s) M = fmaxf(M, pml[2 * s]);
    float lt = 0.f, ot = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float ms = pml[2 * s];
        if (ms > -INFINITY) {
            const float f = exp2f(ms - M);
            lt = fmaf(pml[2 * s + 1], f, lt);
            ot = fmaf(po[(int64_t)s * D + d], f, ot);
        }
    }
    o[(int64_t)bh * D + d] = __float2bfloat16_rn(ot / lt);
    if (lse && d == 0) lse[bh] = (M + log2f(lt)) * 0.6931471805599453f;
}

template <int D>
static cudaError_t decode_bf16_t(const void* q, const void* kn, const void* vn, void* kc, void* vc, void* o,
                                 float* lse, int BH, int cap, int cache_len, const int32_t* lens, int H, float scale,
                                 void* ws, const Paging& pg, cudaStream_t st, const RopeArgs& rope) {
    const int total = cache_len + 1;
    const int splits = decode_num_splits(BH, total);
    int split_len = (total + splits - 1) / splits;
    split_len = (split_len + 15) / 16 * 16;
    const float scale_log2 = scale * 1.4426950408889634f;
    if (pg.table)
        decode_splitkv_kernel<D, true><<<BH * splits, DEC_WARPS * 32, 0, st>>>(
            static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(kn),
            static_cast<const __nv_bfloat16*>(vn), static_cast<__nv_bfloat16*>(kc), static_cast<__nv_bfloat16*>(vc),
            static_cast<__nv_bfloat16*>(o), lse, static_cast<float*>(ws), BH, cap, cache_len, lens, H, splits, split_len,
            scale_log2, pg, rope);
    else
        decode_splitkv_kernel<D, false><<<BH * splits, DEC_WARPS * 32, 0, st>>>(
            static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(kn),
            static_cast<const __nv_bfloat16*>(vn), static_cast<__nv_bfloat16*>(kc), static_cast<__nv_bfloat16*>(vc),
            static_cast<__nv_bfloat16*>(o), lse, static_cast<float*>(ws), BH, cap, cache_len, lens, H, splits, split_len,
            scale_log2, pg, rope);
    count_launches(1);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || splits == 1) return e;
    decode_merge_kernel<D><<<BH, D, 0, st>>>(static_cast<const float*>(ws), static_cast<__nv_bfloat16*>(o), lse,
                                             splits);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_decode_bf16(const void* q, const void* k_new, const void* v_new, void* k_cache,
                               void* v_cache, void* o, float* lse, int B, int H, int D, int cap, int cache_len,
                               const int32_t* lens, float scale, void* ws, const Paging& pg, cudaStream_t st,
                               const RopeArgs& rope) {
    const int BH = B * H;
    return D == 64 ? decode_bf16_t<64>(q, k_new, v_new, k_cache, v_cache, o, lse, BH, cap, cache_len, lens, H, scale, ws, pg, st, rope)
                   : decode_bf16_t<128>(q, k_new, v_new, k_cache, v_cache, o, lse, BH, cap, cache_len, lens, H, scale, ws,
                                        pg, st, rope);
}

// ---------------------------------------------------------------------------
// Built-in scratch for loma_decode_attn_static: the split partials live in this
// fixed array instead of a caller-provided workspace.  In host code the name
// below is only a handle; the device address is looked up per device.
constexpr size_t DEC_STATIC_SCRATCH_BYTES = 8u << 20;   // 8 MiB, held by every device that loads the library
static __device__ __align__(256) unsigned char g_decode_scratch[DEC_STATIC_SCRATCH_BYTES];

size_t decode_static_scratch_bytes() { return DEC_STATIC_SCRATCH_BYTES; }

// Device address of g_decode_scratch on the current device (looked up once per
// device, with that device current).  nullptr if the lookup fails.
static void* decode_static_scratch() {
    static void* addr[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_decode_scratch) != cudaSuccess) return nullptr;
        addr[dev] = p;
    }
    return addr[dev];
}

// Same kernels as launch_decode_bf16, with the partials in the built-in array.
// The caller has checked that decode_workspace_bytes(...) fits.
cudaError_t launch_decode_bf16_static(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                      void* v_cache, void* o, float* lse, int B, int H, int D, int cap,
                                      int cache_len, float scale, cudaStream_t st) {
    void* ws = decode_static_scratch();
    if (!ws) return cudaErrorInvalidSymbol;
    return launch_decode_bf16(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_len, nullptr, scale, ws, Paging{}, st);
}

}  // namespace loma
