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
// One warp per row; a lane owns the pairs (2 lane', 2 lane' + 1) and walks the (batch, head) pairs
// of its slice of the grid.  HBM-bound: Q and K are read and written once.
#include <math.h>

#include "loma_internal.cuh"

namespace loma {

template <typename T>
struct Pair2;   // two adjacent elements <-> two floats
template <>
struct Pair2<float> {
    using V = float2;
    static __device__ __forceinline__ void unpack(const V& v, float& a, float& b) { a = v.x; b = v.y; }
    static __device__ __forceinline__ V pack(float a, float b) { return make_float2(a, b); }
};
template <>
struct Pair2<__nv_bfloat16> {
    using V = uint32_t;
    static __device__ __forceinline__ void unpack(const V& v, float& a, float& b) { a = bf16lo(v); b = bf16hi(v); }
    static __device__ __forceinline__ V pack(float a, float b) { return pack_bf16(a, b); }
};

constexpr int ROPE_WARPS = 8;

template <typename T, int D>
__global__ void __launch_bounds__(ROPE_WARPS * 32)
rope_kernel(T* __restrict__ q, T* __restrict__ k, int BH, int H, Layout L, int64_t sb, int64_t sh, int64_t ss, double log2_base,
            int position_type) {
    using P = Pair2<T>;
    using V = typename P::V;
    constexpr int HALF = D / 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * ROPE_WARPS + warp;
    if (i >= L.S) return;
    const RowInfo r = layout_row(i, L.n_chunks, L.c, L.t, L.s);
    int pos = r.pos;
    if (position_type == 1 && r.zone == LOMA_ZONE_MEM) pos = r.chunk * L.t + r.offset;
    const int d0 = 2 * lane;                // this lane rotates (d0, d0 + HALF) and (d0 + 1, d0 + 1 + HALF)
    const bool active = d0 < HALF;          // D = 64 leaves lanes 16-31 idle
    float cs[2] = {1.f, 1.f}, sn[2] = {0.f, 0.f};
    if (active) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const double theta = exp2(-log2_base * (2.0 * (d0 + u) / D));
            double s_, c_;
            sincos((double)pos * theta, &s_, &c_);
            cs[u] = (float)c_;
            sn[u] = (float)s_;
        }
    }
    if (!active) return;
    const int per = (BH + gridDim.y - 1) / gridDim.y;
    const int bh0 = blockIdx.y * per, bh1 = min(BH, bh0 + per);
    for (int which = 0; which < 2; ++which) {
        T* base = which == 0 ? q : k;
        if (!base) continue;
#pragma unroll 4
        for (int bh = bh0; bh < bh1; ++bh) {
            const int b = bh / H, h = bh - b * H;
            T* row = base + (int64_t)b * sb + (int64_t)h * sh + (int64_t)i * ss;
            V* lo = reinterpret_cast<V*>(row + d0);
            V* hi = reinterpret_cast<V*>(row + d0 + HALF);
            const V vl = *lo, vh = *hi;
            float a0, a1, b0, b1;
            P::unpack(vl, a0, a1);
            P::unpack(vh, b0, b1);
            *lo = P::pack(a0 * cs[0] - b0 * sn[0], a1 * cs[1] - b1 * sn[1]);
            *hi = P::pack(b0 * cs[0] + a0 * sn[0], b1 * cs[1] + a1 * sn[1]);
        }
    }
}

template <typename T, int D>
static cudaError_t rope_t(void* q, void* k, int B, int H, const Layout& L, int64_t sb, int64_t sh, int64_t ss, double theta_base,
                          int position_type, cudaStream_t st) {
    const int BH = B * H;
    const int rows_ctas = (L.S + ROPE_WARPS - 1) / ROPE_WARPS;
    // enough CTAs to fill the GPU several times over; every slice recomputes the row's cos/sin
    int slices = 1;
    while (slices < BH && (int64_t)rows_ctas * slices < 148 * 16) slices *= 2;
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
