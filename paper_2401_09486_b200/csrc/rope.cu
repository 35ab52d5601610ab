// Rotary position embedding of Q and K at LoMA's position ids (Section 4.5, Eq. 14).
//
// The paper hands its position ids to a Llama-2 model, whose attention rotates every (q, k) row by
// its position: with half = D/2 and theta_d = base^(-2d/D), d in [0, half),
//     x'[d]        = x[d] cos(p theta_d) - x[d + half] sin(p theta_d)
//     x'[d + half] = x[d + half] cos(p theta_d) + x[d] sin(p theta_d)
// (the pairing (d, d + half) is the one Llama uses; the paper itself does not spell the rotation out).
// p is the row's position id: reading and repetition rows keep the id of the token they carry or
// reproduce, memory row j of chunk y gets y*tc + (j+1)c - 1 (Eq. 14, "intermittent") or, in the
// generator's other setting, y*t + j ("contiguous").  Nothing is read but Q and K: the ids come
// from the row number by the layout's integer arithmetic, and cos/sin are evaluated once per
// (row, d) in double precision (p reaches tens of thousands, where a float angle has lost the
// digits the 1e-5 bar needs) and reused for every (batch, head).
//
// A lane owns 16 bytes of a row's first half and the partner 16 bytes of its second half and walks
// the (batch, head) pairs of its slice of the grid.  HBM-bound: Q and K are read and written once.
#include <math.h>

#include "loma_internal.cuh"

namespace loma {

template <typename T>
struct Vec16;   // 16 bytes of adjacent elements <-> floats
template <>
struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&x)[4]) {
        return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
    }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&x)[8]) {
        x[0] = bf16lo(v.x); x[1] = bf16hi(v.x); x[2] = bf16lo(v.y); x[3] = bf16hi(v.y);
        x[4] = bf16lo(v.z); x[5] = bf16hi(v.z); x[6] = bf16lo(v.w); x[7] = bf16hi(v.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&x)[8]) {
        return make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]), pack_bf16(x[6], x[7]));
    }
};

constexpr int ROPE_WARPS = 8;

// A lane owns N = 16 / sizeof(T) adjacent features d0.. of the first half and their partners d0 + D/2..
// (two 16-byte accesses per row and tensor); D/2 / N lanes cover a row, so a warp takes 32 N / (D/2) rows.
template <typename T, int D>
__global__ void __launch_bounds__(ROPE_WARPS * 32)
rope_kernel(T* __restrict__ q, T* __restrict__ k, int BH, int H, Layout L, int64_t sb, int64_t sh, int64_t ss, double log2_base,
            int position_type) {
    using V = Vec16<T>;
    constexpr int N = V::N, HALF = D / 2, LPR = HALF / N, RPW = 32 / LPR;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = (blockIdx.x * ROPE_WARPS + warp) * RPW + lane / LPR;
    if (i >= L.S) return;
    const RowInfo r = layout_row(i, L.n_chunks, L.c, L.t, L.s);
    int pos = r.pos;
    if ((position_type & 1) && r.zone == LOMA_ZONE_MEM) pos = r.chunk * L.t + r.offset;
    if (position_type & LOMA_ROPE_INVERSE) pos = -pos;      // the transposed rotation: what a gradient needs on its way back
    const int d0 = (lane % LPR) * N;
    float cs[N], sn[N];
#pragma unroll
    for (int u = 0; u < N; ++u) {
        const double theta = exp2(-log2_base * (2.0 * (d0 + u) / D));
        double s_, c_;
        sincos((double)pos * theta, &s_, &c_);
        cs[u] = (float)c_;
        sn[u] = (float)s_;
    }
    const int per = (BH + gridDim.y - 1) / gridDim.y;
    const int bh0 = blockIdx.y * per, bh1 = min(BH, bh0 + per);
    for (int which = 0; which < 2; ++which) {
        T* base = which == 0 ? q : k;
        if (!base) continue;
#pragma unroll 4
        for (int bh = bh0; bh < bh1; ++bh) {
            const int b = bh / H, h = bh - b * H;
            T* row = base + (int64_t)b * sb + (int64_t)h * sh + (int64_t)i * ss;
            uint4* lo = reinterpret_cast<uint4*>(row + d0);
            uint4* hi = reinterpret_cast<uint4*>(row + d0 + HALF);
            float a[N], c[N], ra[N], rc[N];
            V::unpack(*lo, a);
            V::unpack(*hi, c);
#pragma unroll
            for (int u = 0; u < N; ++u) {
                ra[u] = a[u] * cs[u] - c[u] * sn[u];
                rc[u] = c[u] * cs[u] + a[u] * sn[u];
            }
            *lo = V::pack(ra);
            *hi = V::pack(rc);
        }
    }
}

template <typename T, int D>
static cudaError_t rope_t(void* q, void* k, int B, int H, const Layout& L, int64_t sb, int64_t sh, int64_t ss, double theta_base,
                          int position_type, cudaStream_t st) {
    const int BH = B * H;
    constexpr int RPW = 32 / ((D / 2) / Vec16<T>::N);
    const int rows_ctas = (L.S + ROPE_WARPS * RPW - 1) / (ROPE_WARPS * RPW);
    // enough CTAs to fill the GPU several times over; every slice recomputes its rows' cos/sin
    int slices = 1;
    while (slices < BH && (int64_t)rows_ctas * slices < 148 * 6) slices *= 2;
    if (slices > BH) slices = BH;
    dim3 grid(rows_ctas, slices);
    rope_kernel<T, D><<<grid, ROPE_WARPS * 32, 0, st>>>(static_cast<T*>(q), static_cast<T*>(k), BH, H, L, sb, sh, ss,
                                                        log2(theta_base), position_type);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_rope(void* q, void* k, int B, int H, int D, const Layout& L, int64_t sb, int64_t sh, int64_t ss,
                        loma_dtype dt, double theta_base, int position_type, cudaStream_t st) {
    if (dt == LOMA_F32)
        return D == 64 ? rope_t<float, 64>(q, k, B, H, L, sb, sh, ss, theta_base, position_type, st)
                       : rope_t<float, 128>(q, k, B, H, L, sb, sh, ss, theta_base, position_type, st);
    return D == 64 ? rope_t<__nv_bfloat16, 64>(q, k, B, H, L, sb, sh, ss, theta_base, position_type, st)
                   : rope_t<__nv_bfloat16, 128>(q, k, B, H, L, sb, sh, ss, theta_base, position_type, st);
}

}  // namespace loma
