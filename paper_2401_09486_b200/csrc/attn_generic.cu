// Plain CUDA-core attention kernels: one warp per query row, fp32 arithmetic.
//
// These serve three purposes: the fp32 path (tensor cores would cost mantissa
// bits the 1e-5 bar does not allow), geometries the tensor-core kernels do not
// cover, and an on-GPU second opinion (LOMA_FLAG_FORCE_GENERIC).
//
// Every row of Eq. 7 is an independent softmax over the keys its mask row
// allows.  For each kind of row those keys form a short list of contiguous
// ranges, so a row is described by a count of visible keys and a map from a
// "visible index" to a key pointer -- the mask of Eq. 1-3 is never stored:
//   reading row (y, o):    memory zones of chunks 0..y-1, then own reading
//                          zone up to and including o            (Eq. 1 L, Eq. 3)
//   memory row (y, j):     own reading zone and own memory zone  (Eq. 1 row 2)
//                          [+ earlier memory zones with the prior-memory flag]
//   repetition row (y, o): own memory zone, then itself          (Eq. 1 row 3)
//   decode:                cache[0, len) then the new token      (Appendix A)
//   compress:              cache tail (tc) then the t own keys   (Appendix A)
//   prefill row i:         cache[0, len + i + 1): the cached entries and the new tokens
//                          up to itself, already appended            (Appendix A)
#include <math.h>

#include "loma_internal.cuh"

namespace loma {

// ---------------------------------------------------------------- element IO
template <typename T>
struct Io;

template <>
struct Io<float> {
    // dot of a D-float row in shared memory with a D-element global row
    template <int D>
    static __device__ __forceinline__ float dot(const float* __restrict__ qs, const float* kp) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        const float4* k4 = reinterpret_cast<const float4*>(kp);
        const float4* q4 = reinterpret_cast<const float4*>(qs);
#pragma unroll
        for (int i = 0; i < D / 4; ++i) {
            const float4 kv = k4[i];   // (plain loads: a key row may also sit in shared memory, see the fused rotary embedding)
            const float4 qv = q4[i];
            a0 = fmaf(qv.x, kv.x, a0);
            a1 = fmaf(qv.y, kv.y, a1);
            a2 = fmaf(qv.z, kv.z, a2);
            a3 = fmaf(qv.w, kv.w, a3);
        }
        return (a0 + a1) + (a2 + a3);
    }
    template <int N>
    static __device__ __forceinline__ void load(const float* p, float (&x)[N]) {
#pragma unroll
        for (int i = 0; i < N; ++i) x[i] = p[i];
    }
    template <int N>
    static __device__ __forceinline__ void store(float* p, const float (&x)[N]) {
#pragma unroll
        for (int i = 0; i < N; ++i) p[i] = x[i];
    }
};

template <>
struct Io<__nv_bfloat16> {
    template <int D>
    static __device__ __forceinline__ float dot(const float* __restrict__ qs,
                                                const __nv_bfloat16* kp) {
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        const uint4* k8 = reinterpret_cast<const uint4*>(kp);
        const float4* q4 = reinterpret_cast<const float4*>(qs);
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            const uint4 kv = k8[i];
            const float4 qa = q4[2 * i], qb = q4[2 * i + 1];
            a0 = fmaf(qa.x, bf16lo(kv.x), a0);
            a1 = fmaf(qa.y, bf16hi(kv.x), a1);
            a2 = fmaf(qa.z, bf16lo(kv.y), a2);
            a3 = fmaf(qa.w, bf16hi(kv.y), a3);
            a0 = fmaf(qb.x, bf16lo(kv.z), a0);
            a1 = fmaf(qb.y, bf16hi(kv.z), a1);
            a2 = fmaf(qb.z, bf16lo(kv.w), a2);
            a3 = fmaf(qb.w, bf16hi(kv.w), a3);
        }
        return (a0 + a1) + (a2 + a3);
    }
    template <int N>
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&x)[N]) {
        static_assert(N % 2 == 0, "pairs");
        const uint32_t* u = reinterpret_cast<const uint32_t*>(p);
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            const uint32_t w = u[i];
            x[2 * i] = bf16lo(w);
            x[2 * i + 1] = bf16hi(w);
        }
    }
    template <int N>
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&x)[N]) {
        uint32_t* u = reinterpret_cast<uint32_t*>(p);
#pragma unroll
        for (int i = 0; i < N / 2; ++i) u[i] = pack_bf16(x[2 * i], x[2 * i + 1]);
    }
};

// ------------------------------------------------------------ one query row
// qs: the row's query as D floats in shared memory (this warp's slice).
// map.kptr(v) / map.vptr(v): pointer to the D-element key / value row of
// visible index v, 0 <= v < nkeys.  Online softmax over blocks of 32 keys:
// lane = key for the scores, lane = slice of D for the output.
template <typename T, int D, typename Map>
__device__ __forceinline__ void attend_row(const float* qs, const Map& map, int nkeys, float scale,
                                           T* o_out, float* lse_out, int lane) {
    constexpr int DPL = D / 32;
    float o[DPL];
#pragma unroll
    for (int d = 0; d < DPL; ++d) o[d] = 0.f;
    float m = -INFINITY, l = 0.f;
    for (int base = 0; base < nkeys; base += 32) {
        const int v = base + lane;
        const bool valid = v < nkeys;
        float sc = -INFINITY;
        if (valid) sc = Io<T>::template dot<D>(qs, map.kptr(v)) * scale;
        const float m_new = fmaxf(m, warp_max(sc));
        const float p = valid ? expf(sc - m_new) : 0.f;
        const float alpha = expf(m - m_new);   // first block: exp(-inf) = 0
        l = l * alpha + warp_sum(p);
#pragma unroll
        for (int d = 0; d < DPL; ++d) o[d] *= alpha;
        const int cnt = min(32, nkeys - base);
        for (int jj = 0; jj < cnt; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
            float vv[DPL];
            Io<T>::template load<DPL>(map.vptr(base + jj) + lane * DPL, vv);
#pragma unroll
            for (int d = 0; d < DPL; ++d) o[d] = fmaf(pj, vv[d], o[d]);
        }
        m = m_new;
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int d = 0; d < DPL; ++d) o[d] *= inv;
    Io<T>::template store<DPL>(o_out + lane * DPL, o);
    if (lse_out && lane == 0) *lse_out = m + logf(l);
}

template <typename T, int D>
__device__ __forceinline__ void stage_query(float* qs, const T* qrow, int lane) {
    constexpr int DPL = D / 32;
    float x[DPL];
    Io<T>::template load<DPL>(qrow + lane * DPL, x);
#pragma unroll
    for (int d = 0; d < DPL; ++d) qs[lane * DPL + d] = x[d];
    __syncwarp();
}

// ------------------------------------------------------- masked forward map
template <typename T>
struct TrainMap {
    const T* k;
    const T* v;
    int64_t ss;       // row stride (elements)
    int s, tc, t;
    int kind;         // 0: memory zones of chunks < y then rows [lo, ...)   1: rows [lo, lo+n_range) then row `self`
    int n_prior;      // visible memory keys of earlier chunks (kind 0)
    int lo;           // first row of the contiguous range
    int n_range;      // length of the contiguous range (kind 1)
    int self;         // row index of the trailing self key (kind 1)
    __device__ __forceinline__ int64_t row(int vi) const {
        if (kind == 0) {
            if (vi < n_prior) {
                const int x = vi / t;
                return (int64_t)x * s + tc + (vi - x * t);
            }
            return lo + (vi - n_prior);
        }
        return vi < n_range ? lo + vi : self;
    }
    __device__ __forceinline__ const T* kptr(int vi) const { return k + row(vi) * ss; }
    __device__ __forceinline__ const T* vptr(int vi) const { return v + row(vi) * ss; }
};

// (chunk, zone, offset) of row i, as in Section 4.1; the reading tail counts as chunk n_chunks
__device__ __forceinline__ void decompose_row(const Layout& L, int i, int& y, int& zone, int& off) {
    if (L.s == 0 || i >= L.n_chunks * L.s) {
        y = L.n_chunks; zone = LOMA_ZONE_READ; off = i - L.n_chunks * L.s;
    } else {
        y = i / L.s;
        const int r = i - y * L.s;
        if (r < L.tc) { zone = LOMA_ZONE_READ; off = r; }
        else if (r < L.tc + L.t) { zone = LOMA_ZONE_MEM; off = r - L.tc; }
        else { zone = LOMA_ZONE_REP; off = r - L.tc - L.t; }
    }
}

// Fills the visible-key map of row i and returns its number of visible keys.
template <typename T>
__device__ __forceinline__ int train_row_map(const Layout& L, int i, const T* k, const T* v, int64_t ss, TrainMap<T>& map) {
    int y, zone, off;
    decompose_row(L, i, y, zone, off);
    map.k = k; map.v = v; map.ss = ss; map.s = L.s; map.tc = L.tc; map.t = L.t;
    map.n_range = 0; map.self = 0;
    if (zone == LOMA_ZONE_READ) {                 // Eq. 3 reading rows + L of Eq. 1
        map.kind = 0; map.n_prior = y * L.t; map.lo = y * L.s;
        return map.n_prior + off + 1;
    }
    if (zone == LOMA_ZONE_MEM) {                  // Eq. 1 second block row
        map.kind = 0; map.lo = y * L.s;
        map.n_prior = (L.flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM) ? y * L.t : 0;
        return map.n_prior + L.tc + L.t;
    }
    map.kind = 1; map.n_prior = 0; map.lo = y * L.s + L.tc; map.n_range = L.t; map.self = i;   // Eq. 1 third block row
    return L.t + 1;
}

constexpr int GENERIC_WARPS = 8;

template <typename T, int D>
__global__ void __launch_bounds__(GENERIC_WARPS * 32)
masked_attn_generic_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                           T* __restrict__ o, float* __restrict__ lse, int H, Layout L, int64_t sb,
                           int64_t sh, int64_t ss, float scale) {
    __shared__ __align__(16) float q_sh[GENERIC_WARPS][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * GENERIC_WARPS + warp;
    if (i >= L.S) return;
    const int bh = blockIdx.y;
    const int b = bh / H, h = bh - b * H;
    const int64_t base = (int64_t)b * sb + (int64_t)h * sh;

    TrainMap<T> map;
    const int nkeys = train_row_map(L, i, k + base, v + base, ss, map);
    stage_query<T, D>(q_sh[warp], q + base + (int64_t)i * ss, lane);
    attend_row<T, D>(q_sh[warp], map, nkeys, scale, o + base + (int64_t)i * ss,
                     lse ? lse + (int64_t)bh * L.S + i : nullptr, lane);
}

// --------------------------------------------------------------- decode map
template <typename T>
struct DecodeMap {
    const T* kc;
    const T* vc;
    const T* kn;
    const T* vn;
    int len, D;
    Paging pg;        // pg.table != NULL: kc / vc are the pools and slots go through the block table
    int b, h, H;
    __device__ __forceinline__ int64_t slot(int vi) const {
        if (!pg.table) return (int64_t)vi * D;
        const int page = min(max(pg.table[(int64_t)b * pg.max_pages + (vi >> pg.log2_ps)], 0), pg.n_pages - 1);
        return ((((int64_t)page * H + h) << pg.log2_ps) + (vi & ((1 << pg.log2_ps) - 1))) * D;
    }
    __device__ __forceinline__ const T* kptr(int vi) const { return vi < len ? kc + slot(vi) : kn; }
    __device__ __forceinline__ const T* vptr(int vi) const { return vi < len ? vc + slot(vi) : vn; }
};

// to / from the storage type, round to nearest even
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

template <typename T, int D>
__global__ void __launch_bounds__(32)
decode_generic_kernel(const T* __restrict__ q, const T* __restrict__ k_new, const T* __restrict__ v_new,
                      T* __restrict__ k_cache, T* __restrict__ v_cache, T* __restrict__ o,
                      float* __restrict__ lse, int cap, int cache_len_max, const int32_t* __restrict__ lens, int H,
                      float scale, Paging pg, RopeArgs rope) {
    __shared__ __align__(16) float q_sh[D];
    __shared__ __align__(16) T kn_sh[D];       // the new key, rotated (fused rotary embedding only)
    const int bh = blockIdx.x, lane = threadIdx.x;
    const int cache_len = lens ? min(max(lens[bh / H], 0), cache_len_max) : cache_len_max;   // ragged batch
    T* kc = pg.table ? k_cache : k_cache + (int64_t)bh * cap * D;
    T* vc = pg.table ? v_cache : v_cache + (int64_t)bh * cap * D;
    DecodeMap<T> map;
    map.kc = kc; map.vc = vc; map.len = cache_len; map.D = D;
    map.pg = pg; map.b = bh / H; map.h = bh - map.b * H; map.H = H;
    const int64_t new_off = map.slot(cache_len);
    map.kn = k_new ? k_new + (int64_t)bh * D : kc + new_off;
    map.vn = v_new ? v_new + (int64_t)bh * D : vc + new_off;
    stage_query<T, D>(q_sh, q + (int64_t)bh * D, lane);
    if (rope.on) {
        // Section 4.5: q and the new key rotated by the step's position id, here instead of in a pass of their own;
        // the rotated key, rounded to the storage type, is what the step attends to and appends
        const int pos = rope.pos_seq ? rope.pos_seq[bh / H] : rope.pos0;
        for (int d = lane; d < D / 2; d += 32) {
            float c, sn;
            rope_cos_sin(pos, d, D, rope.log2_base, c, sn);
            const float qa = q_sh[d], qb = q_sh[d + D / 2];
            q_sh[d] = qa * c - qb * sn;
            q_sh[d + D / 2] = qb * c + qa * sn;
            const float ka = to_f32(map.kn[d]), kb = to_f32(map.kn[d + D / 2]);
            kn_sh[d] = from_f32<T>(ka * c - kb * sn);
            kn_sh[d + D / 2] = from_f32<T>(kb * c + ka * sn);
        }
        __syncwarp();
        map.kn = kn_sh;
    }
    attend_row<T, D>(q_sh, map, cache_len + 1, scale, o + (int64_t)bh * D, lse ? lse + bh : nullptr, lane);
    if (k_new) {      // append: the slot is read by nobody in this launch
        constexpr int DPL = D / 32;
#pragma unroll
        for (int d = 0; d < DPL; ++d) {
            kc[new_off + lane * DPL + d] = map.kn[lane * DPL + d];
            vc[new_off + lane * DPL + d] = v_new[(int64_t)bh * D + lane * DPL + d];
        }
    }
}

// --------------------------------------------- several new tokens over a cache
// Appendix A, inference_input with l tokens: the mask tril(ones(l, l + len), diagonal = len).  The new
// tokens' K/V have been appended at [len, len + l) by cache_append_kernel before this launch, so row i simply
// sees cache rows 0 .. len + i.
template <typename T>
struct CacheRangeMap {
    const T* kc;   // the (b,h)'s cache (contiguous) or the pool (paged)
    const T* vc;
    int D;
    Paging pg;
    int b, h, H;
    __device__ __forceinline__ int64_t slot(int j) const {
        if (!pg.table) return (int64_t)j * D;
        const int page = min(max(pg.table[(int64_t)b * pg.max_pages + (j >> pg.log2_ps)], 0), pg.n_pages - 1);
        return ((((int64_t)page * H + h) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * D;
    }
    __device__ __forceinline__ const T* kptr(int vi) const { return kc + slot(vi); }
    __device__ __forceinline__ const T* vptr(int vi) const { return vc + slot(vi); }
};

// lens (device, [B], or NULL): every sequence's own number of earlier entries, clamped to [0, cache_len]
template <typename T, int D>
__global__ void __launch_bounds__(GENERIC_WARPS * 32)
prefill_generic_kernel(const T* __restrict__ q, const T* __restrict__ k_cache, const T* __restrict__ v_cache,
                       T* __restrict__ o, float* __restrict__ lse, int l, int cap, int cache_len,
                       const int32_t* __restrict__ lens, int H, Paging pg, float scale) {
    __shared__ __align__(16) float q_sh[GENERIC_WARPS][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * GENERIC_WARPS + warp;
    if (i >= l) return;
    const int bh = blockIdx.y;
    CacheRangeMap<T> map;
    map.b = bh / H; map.h = bh - map.b * H; map.H = H; map.pg = pg; map.D = D;
    map.kc = pg.table ? k_cache : k_cache + (int64_t)bh * cap * D;
    map.vc = pg.table ? v_cache : v_cache + (int64_t)bh * cap * D;
    const int own = lens ? min(max(__ldg(lens + map.b), 0), cache_len) : cache_len;
    const int64_t row = ((int64_t)bh * l + i) * D;
    stage_query<T, D>(q_sh[warp], q + row, lane);
    attend_row<T, D>(q_sh[warp], map, own + i + 1, scale, o + row, lse ? lse + (int64_t)bh * l + i : nullptr, lane);
}

// k_new, v_new [B, H, l, D] -> cache rows [len, len + l) of every (b, h): 16-byte vectors, bit-exact.  With per-sequence
// lengths (pad_to > 1) the rows from the sequence's new end up to the next multiple of pad_to (and at most cap) are
// set to zero as well: the tensor-core kernel multiplies them by probabilities of zero, so they have to be finite, and
// the contents of the cache past the valid length are unspecified anyway.  k_new == NULL: only that.
__global__ void cache_append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                    uint4* __restrict__ k_cache, uint4* __restrict__ v_cache, int vec_per_row, int l, int cap,
                                    int cache_len, const int32_t* __restrict__ lens, int H, Paging pg, int pad_to,
                                    int copy_k) {
    const int bh = blockIdx.y;
    const int b = bh / H, h = bh - b * H;
    const int own = lens ? min(max(__ldg(lens + b), 0), cache_len) : cache_len;
    auto slot = [&](int j) -> int64_t {   // row j of this (b,h) in 16-byte units
        if (!pg.table) return ((int64_t)bh * cap + j) * vec_per_row;
        const int page = min(max(__ldg(pg.table + (int64_t)b * pg.max_pages + (j >> pg.log2_ps)), 0), pg.n_pages - 1);
        return ((((int64_t)page * H + h) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * vec_per_row;
    };
    const int end = own + l;
    const int pad_end = pad_to > 1 ? min((end + pad_to - 1) / pad_to * pad_to, cap) : end;
    const int64_t n = (int64_t)(pad_end - own) * vec_per_row, n_new = (int64_t)l * vec_per_row;
    const int64_t in = (int64_t)bh * n_new;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        const int r = (int)(e / vec_per_row), cv = (int)(e - (int64_t)r * vec_per_row);
        const int64_t out = slot(own + r) + cv;
        if (e < n_new) {
            if (k_new && copy_k) k_cache[out] = __ldg(k_new + in + e);   // (copy_k == 0: the keys arrive rotated, from another kernel)
            if (v_new) v_cache[out] = __ldg(v_new + in + e);
        } else {
            k_cache[out] = make_uint4(0, 0, 0, 0);
            v_cache[out] = make_uint4(0, 0, 0, 0);
        }
    }
}

// Rotary embedding of a prompt piece (Section 4.5; Appendix A, inference_input: new token i of a sequence has the id
// cursor + i): q rotated into q_rot (the caller's output buffer, which the attention kernels then read as their
// query), k_new rotated, rounded to the storage type and written to the cache rows [len, len + l).  One thread per
// feature pair (d, d + D/2).
template <typename T, int D>
__global__ void __launch_bounds__(128)
prefill_rope_kernel(const T* __restrict__ q, const T* __restrict__ k_new, T* __restrict__ q_rot, T* __restrict__ k_cache,
                    int l, int cap, int cache_len, const int32_t* __restrict__ lens, int H, Paging pg, RopeArgs rope) {
    constexpr int HALF = D / 2, RPB = 128 / HALF;      // rows per block
    const int i = blockIdx.x * RPB + threadIdx.x / HALF, d = threadIdx.x % HALF;
    if (i >= l) return;
    const int bh = blockIdx.y, b = bh / H, h = bh - b * H;
    const int own = lens ? min(max(__ldg(lens + b), 0), cache_len) : cache_len;
    const int pos = (rope.pos_seq ? __ldg(rope.pos_seq + b) : rope.pos0) + i * rope.stride;
    float c, sn;
    rope_cos_sin(pos, d, D, rope.log2_base, c, sn);
    const int64_t row = ((int64_t)bh * l + i) * D;
    {
        const float a = to_f32(q[row + d]), bb = to_f32(q[row + d + HALF]);
        q_rot[row + d] = from_f32<T>(a * c - bb * sn);
        q_rot[row + d + HALF] = from_f32<T>(bb * c + a * sn);
    }
    const int j = own + i;
    int64_t out;
    if (!pg.table) {
        out = ((int64_t)bh * cap + j) * D;
    } else {
        const int page = min(max(__ldg(pg.table + (int64_t)b * pg.max_pages + (j >> pg.log2_ps)), 0), pg.n_pages - 1);
        out = ((((int64_t)page * H + h) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * D;
    }
    const float a = to_f32(k_new[row + d]), bb = to_f32(k_new[row + d + HALF]);
    k_cache[out + d] = from_f32<T>(a * c - bb * sn);
    k_cache[out + d + HALF] = from_f32<T>(bb * c + a * sn);
}

// ------------------------------------------------------------- compress map
template <typename T>
struct CompressMap {
    const T* kc;   // the (b,h)'s cache (contiguous) or the pool (paged)
    const T* vc;
    const T* km;   // this (b,h)'s t memory keys
    const T* vm;
    int lo, n_cache, D;   // visible cache slots [lo, lo + n_cache)
    Paging pg;
    int b, h, H;
    __device__ __forceinline__ int64_t slot(int j) const {
        if (!pg.table) return (int64_t)j * D;
        const int page = min(max(pg.table[(int64_t)b * pg.max_pages + (j >> pg.log2_ps)], 0), pg.n_pages - 1);
        return ((((int64_t)page * H + h) << pg.log2_ps) + (j & ((1 << pg.log2_ps) - 1))) * D;
    }
    __device__ __forceinline__ const T* kptr(int vi) const {
        return vi < n_cache ? kc + slot(lo + vi) : km + (int64_t)(vi - n_cache) * D;
    }
    __device__ __forceinline__ const T* vptr(int vi) const {
        return vi < n_cache ? vc + slot(lo + vi) : vm + (int64_t)(vi - n_cache) * D;
    }
};

// One CTA per (b,h): its warps take the t memory rows in turn; after a block
// barrier (every read of the tail by this (b,h) is done, and no other CTA reads
// it) the t memory K/V rows are copied over slots [mem_len, mem_len+t).
template <typename T, int D>
__global__ void __launch_bounds__(GENERIC_WARPS * 32)
compress_generic_kernel(const T* __restrict__ q_mem, const T* __restrict__ k_mem,
                        const T* __restrict__ v_mem, T* __restrict__ k_cache, T* __restrict__ v_cache,
                        T* __restrict__ o_mem, float* __restrict__ lse, int cap, int mem_len, const int32_t* __restrict__ mem_lens,
                        int H, int t, int tc, unsigned flags, float scale, Paging pg, RopeArgs rope) {
    __shared__ __align__(16) float q_sh[GENERIC_WARPS][D];
    extern __shared__ __align__(16) uint8_t km_rot_raw[];   // t x D rotated memory keys (fused rotary embedding only)
    const int bh = blockIdx.x;
    if (mem_lens) {                          // ragged batch: own count of memory entries; negative = not compressing now
        const int own = mem_lens[bh / H];
        if (own < 0) return;
        mem_len = min(own, mem_len);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    T* kc = pg.table ? k_cache : k_cache + (int64_t)bh * cap * D;
    T* vc = pg.table ? v_cache : v_cache + (int64_t)bh * cap * D;
    const int lo = (flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM) ? 0 : mem_len;
    CompressMap<T> map;
    map.kc = kc; map.vc = vc; map.lo = lo;
    map.km = k_mem + (int64_t)bh * t * D; map.vm = v_mem + (int64_t)bh * t * D;
    map.n_cache = mem_len + tc - lo; map.D = D;
    map.pg = pg; map.b = bh / H; map.h = bh - map.b * H; map.H = H;
    const int rope_pos0 = rope.pos_seq ? rope.pos_seq[bh / H] : rope.pos0;
    if (rope.on) {
        // Section 4.5: memory row j is rotated by the id pos0 + j * stride; its key, rounded to the storage type,
        // is what every memory query attends to and what goes into the cache
        T* km_rot = reinterpret_cast<T*>(km_rot_raw);
        for (int e = threadIdx.x; e < t * (D / 2); e += blockDim.x) {
            const int j = e / (D / 2), d = e - j * (D / 2);
            float c, sn;
            rope_cos_sin(rope_pos0 + j * rope.stride, d, D, rope.log2_base, c, sn);
            const float a = to_f32(map.km[(int64_t)j * D + d]), b = to_f32(map.km[(int64_t)j * D + d + D / 2]);
            km_rot[j * D + d] = from_f32<T>(a * c - b * sn);
            km_rot[j * D + d + D / 2] = from_f32<T>(b * c + a * sn);
        }
        __syncthreads();
        map.km = km_rot;
    }
    for (int j = warp; j < t; j += GENERIC_WARPS) {
        stage_query<T, D>(q_sh[warp], q_mem + ((int64_t)bh * t + j) * D, lane);
        if (rope.on) {
            for (int d = lane; d < D / 2; d += 32) {
                float c, sn;
                rope_cos_sin(rope_pos0 + j * rope.stride, d, D, rope.log2_base, c, sn);
                const float a = q_sh[warp][d], b = q_sh[warp][d + D / 2];
                q_sh[warp][d] = a * c - b * sn;
                q_sh[warp][d + D / 2] = b * c + a * sn;
            }
            __syncwarp();
        }
        attend_row<T, D>(q_sh[warp], map, map.n_cache + t, scale, o_mem + ((int64_t)bh * t + j) * D,
                         lse ? lse + (int64_t)bh * t + j : nullptr, lane);
        __syncwarp();
    }
    __syncthreads();
    // compaction: 16-byte vector copies, bit for bit
    constexpr int VEC = 16 / sizeof(T);
    constexpr int VPR = D / VEC;             // 16-byte vectors per row
    const uint4* ksrc = reinterpret_cast<const uint4*>(map.km);
    const uint4* vsrc = reinterpret_cast<const uint4*>(map.vm);
    for (int e = threadIdx.x; e < t * VPR; e += blockDim.x) {
        const int r = e / VPR, cv = e - r * VPR;
        const int64_t off = map.slot(mem_len + r) + cv * VEC;
        *reinterpret_cast<uint4*>(kc + off) = ksrc[e];
        *reinterpret_cast<uint4*>(vc + off) = vsrc[e];
    }
}

// ------------------------------------------------------------ masked backward
// Gradients of Eq. 7 (Section 4.4).  With P_ij = exp(scale q_i.k_j - lse_i) on the allowed
// entries, delta_i = dO_i . O_i (= sum_j P_ij dP_ij) and dA_ij = P_ij (dO_i . v_j - delta_i):
//   dQ_i = scale sum_j dA_ij k_j     one warp per query row, over the keys the row sees
//   dK_j = scale sum_i dA_ij q_i     one warp per key row, over the rows that see the key
//   dV_j =       sum_i P_ij dO_i
// Each output row is owned by one warp: no atomics, results repeat bit for bit.
template <typename T, int D>
__global__ void __launch_bounds__(GENERIC_WARPS * 32)
masked_attn_bwd_dq_generic_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                  const T* __restrict__ o, const T* __restrict__ d_o, const float* __restrict__ lse,
                                  T* __restrict__ dq, float* __restrict__ delta, int H, Layout L, int64_t sb, int64_t sh,
                                  int64_t ss, float scale) {
    __shared__ __align__(16) float q_sh[GENERIC_WARPS][D];
    __shared__ __align__(16) float g_sh[GENERIC_WARPS][D];
    constexpr int DPL = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * GENERIC_WARPS + warp;
    if (i >= L.S) return;
    const int bh = blockIdx.y;
    const int b = bh / H, h = bh - b * H;
    const int64_t base = (int64_t)b * sb + (int64_t)h * sh;
    TrainMap<T> map;
    const int nkeys = train_row_map(L, i, k + base, v + base, ss, map);
    stage_query<T, D>(q_sh[warp], q + base + (int64_t)i * ss, lane);
    stage_query<T, D>(g_sh[warp], d_o + base + (int64_t)i * ss, lane);
    float dl;
    {
        float ov[DPL];
        Io<T>::template load<DPL>(o + base + (int64_t)i * ss + lane * DPL, ov);
        float part = 0.f;
#pragma unroll
        for (int d = 0; d < DPL; ++d) part = fmaf(g_sh[warp][lane * DPL + d], ov[d], part);
        dl = warp_sum(part);
        if (lane == 0) delta[(int64_t)bh * L.S + i] = dl;
    }
    const float lse_i = lse[(int64_t)bh * L.S + i];
    float acc[DPL];
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc[d] = 0.f;
    for (int kb = 0; kb < nkeys; kb += 32) {
        const int vi = kb + lane;
        float da = 0.f;
        if (vi < nkeys) {
            const float sc = Io<T>::template dot<D>(q_sh[warp], map.kptr(vi)) * scale;
            const float p = expf(sc - lse_i);
            const float dp = Io<T>::template dot<D>(g_sh[warp], map.vptr(vi));
            da = p * (dp - dl);
        }
        const int cnt = min(32, nkeys - kb);
        for (int jj = 0; jj < cnt; ++jj) {
            const float dj = __shfl_sync(0xffffffffu, da, jj);
            float kk[DPL];
            Io<T>::template load<DPL>(map.kptr(kb + jj) + lane * DPL, kk);
#pragma unroll
            for (int d = 0; d < DPL; ++d) acc[d] = fmaf(dj, kk[d], acc[d]);
        }
    }
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc[d] *= scale;
    Io<T>::template store<DPL>(dq + base + (int64_t)i * ss + lane * DPL, acc);
}

// Rows that see key j, as a visible index -> row map (the columns of Eq. 2 read downwards):
//   reading key (y, o):    reading rows o.. of chunk y, then the chunk's memory rows (contiguous)
//   memory key (y, j):     memory and repetition rows of chunk y (contiguous), then the reading
//                          rows [and, with the prior-memory flag, memory rows] of every later
//                          chunk, then the reading tail
//   repetition key:        its own row
struct SeenByMap {
    int lo, n_first;      // first contiguous range
    int y_next, seg_len;  // later chunks y_next.. contribute rows [y*s, y*s + seg_len)
    int n_later, s, tail0;
    __device__ __forceinline__ int row(int vi) const {
        if (vi < n_first) return lo + vi;
        vi -= n_first;
        if (vi < n_later) {
            const int x = vi / seg_len;
            return (y_next + x) * s + (vi - x * seg_len);
        }
        return tail0 + (vi - n_later);
    }
};

__device__ __forceinline__ int seen_by_map(const Layout& L, int j, SeenByMap& m) {
    int y, zone, off;
    decompose_row(L, j, y, zone, off);
    m.s = L.s; m.tail0 = L.n_chunks * L.s; m.n_later = 0; m.seg_len = 1; m.y_next = 0;
    if (zone == LOMA_ZONE_READ) {
        m.lo = j;
        m.n_first = (y == L.n_chunks) ? L.S - j : (L.tc - off) + L.t;
        return m.n_first;
    }
    if (zone == LOMA_ZONE_REP) { m.lo = j; m.n_first = 1; return 1; }
    m.lo = y * L.s + L.tc;
    m.n_first = (y + 1) * L.s - m.lo;
    m.y_next = y + 1;
    m.seg_len = L.tc + ((L.flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM) ? L.t : 0);
    m.n_later = (L.n_chunks - 1 - y) * m.seg_len;
    return m.n_first + m.n_later + L.tail_read;
}

template <typename T, int D>
__global__ void __launch_bounds__(GENERIC_WARPS * 32)
masked_attn_bwd_dkv_generic_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                   const T* __restrict__ d_o, const float* __restrict__ lse,
                                   const float* __restrict__ delta, T* __restrict__ dk, T* __restrict__ dv, int H,
                                   Layout L, int64_t sb, int64_t sh, int64_t ss, float scale) {
    __shared__ __align__(16) float k_sh[GENERIC_WARPS][D];
    __shared__ __align__(16) float v_sh[GENERIC_WARPS][D];
    constexpr int DPL = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * GENERIC_WARPS + warp;
    if (j >= L.S) return;
    const int bh = blockIdx.y;
    const int b = bh / H, h = bh - b * H;
    const int64_t base = (int64_t)b * sb + (int64_t)h * sh;
    SeenByMap map;
    const int nrows = seen_by_map(L, j, map);
    stage_query<T, D>(k_sh[warp], k + base + (int64_t)j * ss, lane);
    stage_query<T, D>(v_sh[warp], v + base + (int64_t)j * ss, lane);
    float acc_k[DPL], acc_v[DPL];
#pragma unroll
    for (int d = 0; d < DPL; ++d) { acc_k[d] = 0.f; acc_v[d] = 0.f; }
    for (int rb = 0; rb < nrows; rb += 32) {
        const int vi = rb + lane;
        float p = 0.f, da = 0.f;
        int i = 0;
        if (vi < nrows) {
            i = map.row(vi);
            const float sc = Io<T>::template dot<D>(k_sh[warp], q + base + (int64_t)i * ss) * scale;
            p = expf(sc - lse[(int64_t)bh * L.S + i]);
            const float dp = Io<T>::template dot<D>(v_sh[warp], d_o + base + (int64_t)i * ss);
            da = p * (dp - delta[(int64_t)bh * L.S + i]);
        }
        const int cnt = min(32, nrows - rb);
        for (int jj = 0; jj < cnt; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
            const float dj = __shfl_sync(0xffffffffu, da, jj);
            const int ii = __shfl_sync(0xffffffffu, i, jj);
            float qq[DPL], gg[DPL];
            Io<T>::template load<DPL>(q + base + (int64_t)ii * ss + lane * DPL, qq);
            Io<T>::template load<DPL>(d_o + base + (int64_t)ii * ss + lane * DPL, gg);
#pragma unroll
            for (int d = 0; d < DPL; ++d) {
                acc_k[d] = fmaf(dj, qq[d], acc_k[d]);
                acc_v[d] = fmaf(pj, gg[d], acc_v[d]);
            }
        }
    }
#pragma unroll
    for (int d = 0; d < DPL; ++d) acc_k[d] *= scale;
    Io<T>::template store<DPL>(dk + base + (int64_t)j * ss + lane * DPL, acc_k);
    Io<T>::template store<DPL>(dv + base + (int64_t)j * ss + lane * DPL, acc_v);
}

// ------------------------------------------------------------------ launchers
template <typename T, int D>
static cudaError_t masked_generic_t(const void* q, const void* k, const void* v, void* o, float* lse, int B,
                                    int H, const Layout& L, int64_t sb, int64_t sh, int64_t ss, float scale,
                                    cudaStream_t st) {
    dim3 grid((L.S + GENERIC_WARPS - 1) / GENERIC_WARPS, B * H);
    masked_attn_generic_kernel<T, D><<<grid, GENERIC_WARPS * 32, 0, st>>>(
        static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<T*>(o), lse,
        H, L, sb, sh, ss, scale);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_masked_attn_generic(const void* q, const void* k, const void* v, void* o, float* lse,
                                       int B, int H, int D, const Layout& L, int64_t sb, int64_t sh,
                                       int64_t ss, loma_dtype dt, float scale, cudaStream_t st) {
    if (dt == LOMA_F32) {
        return D == 64 ? masked_generic_t<float, 64>(q, k, v, o, lse, B, H, L, sb, sh, ss, scale, st)
                       : masked_generic_t<float, 128>(q, k, v, o, lse, B, H, L, sb, sh, ss, scale, st);
    }
    return D == 64 ? masked_generic_t<__nv_bfloat16, 64>(q, k, v, o, lse, B, H, L, sb, sh, ss, scale, st)
                   : masked_generic_t<__nv_bfloat16, 128>(q, k, v, o, lse, B, H, L, sb, sh, ss, scale, st);
}

template <typename T, int D>
static cudaError_t masked_bwd_generic_t(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                        const float* lse, void* dq, void* dk, void* dv, float* delta, int B, int H,
                                        const Layout& L, int64_t sb, int64_t sh, int64_t ss, float scale,
                                        int parts, cudaStream_t st) {
    dim3 grid((L.S + GENERIC_WARPS - 1) / GENERIC_WARPS, B * H);
    if (parts & 1)
        masked_attn_bwd_dq_generic_kernel<T, D><<<grid, GENERIC_WARPS * 32, 0, st>>>(
            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<const T*>(o),
            static_cast<const T*>(d_o), lse, static_cast<T*>(dq), delta, H, L, sb, sh, ss, scale);
    if (parts & 2)
        masked_attn_bwd_dkv_generic_kernel<T, D><<<grid, GENERIC_WARPS * 32, 0, st>>>(
            static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<const T*>(d_o), lse,
            delta, static_cast<T*>(dk), static_cast<T*>(dv), H, L, sb, sh, ss, scale);
    count_launches((parts & 1) + ((parts >> 1) & 1));
    return cudaGetLastError();
}

cudaError_t launch_masked_attn_bwd_generic(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                           const float* lse, void* dq, void* dk, void* dv, float* delta, int B, int H,
                                           int D, const Layout& L, int64_t sb, int64_t sh, int64_t ss, loma_dtype dt,
                                           float scale, int parts, cudaStream_t st) {
    if (dt == LOMA_F32) {
        return D == 64 ? masked_bwd_generic_t<float, 64>(q, k, v, o, d_o, lse, dq, dk, dv, delta, B, H, L, sb, sh, ss, scale, parts, st)
                       : masked_bwd_generic_t<float, 128>(q, k, v, o, d_o, lse, dq, dk, dv, delta, B, H, L, sb, sh, ss, scale, parts, st);
    }
    return D == 64 ? masked_bwd_generic_t<__nv_bfloat16, 64>(q, k, v, o, d_o, lse, dq, dk, dv, delta, B, H, L, sb, sh, ss, scale, parts, st)
                   : masked_bwd_generic_t<__nv_bfloat16, 128>(q, k, v, o, d_o, lse, dq, dk, dv, delta, B, H, L, sb, sh, ss, scale, parts, st);
}

template <typename T, int D>
static cudaError_t decode_generic_t(const void* q, const void* kn, const void* vn, void* kc, void* vc,
                                    void* o, float* lse, int BH, int cap, int cache_len, const int32_t* lens, int H,
                                    float scale, const Paging& pg, cudaStream_t st, const RopeArgs& rope) {
    decode_generic_kernel<T, D><<<BH, 32, 0, st>>>(static_cast<const T*>(q), static_cast<const T*>(kn),
                                                   static_cast<const T*>(vn), static_cast<T*>(kc),
                                                   static_cast<T*>(vc), static_cast<T*>(o), lse, cap,
                                                   cache_len, lens, H, scale, pg, rope);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_decode_generic(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                  void* v_cache, void* o, float* lse, int B, int H, int D, int cap,
                                  int cache_len, const int32_t* lens, loma_dtype dt, float scale, const Paging& pg,
                                  cudaStream_t st, const RopeArgs& rope) {
    const int BH = B * H;
    if (dt == LOMA_F32) {
        return D == 64 ? decode_generic_t<float, 64>(q, k_new, v_new, k_cache, v_cache, o, lse, BH, cap,
                                                     cache_len, lens, H, scale, pg, st, rope)
                       : decode_generic_t<float, 128>(q, k_new, v_new, k_cache, v_cache, o, lse, BH, cap,
                                                      cache_len, lens, H, scale, pg, st, rope);
    }
    return D == 64 ? decode_generic_t<__nv_bfloat16, 64>(q, k_new, v_new, k_cache, v_cache, o, lse, BH, cap,
                                                         cache_len, lens, H, scale, pg, st, rope)
                   : decode_generic_t<__nv_bfloat16, 128>(q, k_new, v_new, k_cache, v_cache, o, lse, BH, cap,
                                                          cache_len, lens, H, scale, pg, st, rope);
}

template <typename T, int D>
static cudaError_t compress_generic_t(const void* qm, const void* km, const void* vm, void* kc, void* vc,
                                      void* om, float* lse, int BH, int cap, int mem_len, const int32_t* mem_lens, int H, int t,
                                      int tc, unsigned flags, float scale, const Paging& pg, cudaStream_t st,
                                      const RopeArgs& rope) {
    const size_t dyn = rope.on ? (size_t)t * D * sizeof(T) : 0;
    if (dyn > 48 * 1024) {
        if (dyn > 200 * 1024) return cudaErrorNotSupported;
        const cudaError_t ea = cudaFuncSetAttribute(compress_generic_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
        if (ea != cudaSuccess) return ea;
    }
    compress_generic_kernel<T, D><<<BH, GENERIC_WARPS * 32, dyn, st>>>(
        static_cast<const T*>(qm), static_cast<const T*>(km), static_cast<const T*>(vm), static_cast<T*>(kc),
        static_cast<T*>(vc), static_cast<T*>(om), lse, cap, mem_len, mem_lens, H, t, tc, flags, scale, pg, rope);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_compress_generic(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache,
                                    void* v_cache, void* o_mem, float* lse, int B, int H, int D, int cap,
                                    int mem_len, const int32_t* mem_lens, int c, int t, loma_dtype dt, float scale,
                                    unsigned flags, const Paging& pg, cudaStream_t st, const RopeArgs& rope) {
    const int BH = B * H, tc = c * t;
    if (dt == LOMA_F32) {
        return D == 64 ? compress_generic_t<float, 64>(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, BH,
                                                       cap, mem_len, mem_lens, H, t, tc, flags, scale, pg, st, rope)
                       : compress_generic_t<float, 128>(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, BH,
                                                        cap, mem_len, mem_lens, H, t, tc, flags, scale, pg, st, rope);
    }
    return D == 64 ? compress_generic_t<__nv_bfloat16, 64>(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse,
                                                           BH, cap, mem_len, mem_lens, H, t, tc, flags, scale, pg, st, rope)
                   : compress_generic_t<__nv_bfloat16, 128>(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse,
                                                            BH, cap, mem_len, mem_lens, H, t, tc, flags, scale, pg, st, rope);
}

template <typename T, int D>
static cudaError_t prefill_generic_t(const void* q, const void* kc, const void* vc, void* o, float* lse, int BH, int l,
                                     int cap, int cache_len, const int32_t* lens, int H, const Paging& pg, float scale,
                                     cudaStream_t st) {
    dim3 grid((l + GENERIC_WARPS - 1) / GENERIC_WARPS, BH);
    prefill_generic_kernel<T, D><<<grid, GENERIC_WARPS * 32, 0, st>>>(static_cast<const T*>(q), static_cast<const T*>(kc),
                                                                     static_cast<const T*>(vc), static_cast<T*>(o), lse, l, cap,
                                                                     cache_len, lens, H, pg, scale);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_prefill_attn_generic(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                                        int B, int H, int D, int l, int cap, int cache_len, const int32_t* lens,
                                        const Paging& pg, loma_dtype dt, float scale, cudaStream_t st) {
    const int BH = B * H;
    if (dt == LOMA_F32)
        return D == 64 ? prefill_generic_t<float, 64>(q, k_cache, v_cache, o, lse, BH, l, cap, cache_len, lens, H, pg, scale, st)
                       : prefill_generic_t<float, 128>(q, k_cache, v_cache, o, lse, BH, l, cap, cache_len, lens, H, pg, scale, st);
    return D == 64 ? prefill_generic_t<__nv_bfloat16, 64>(q, k_cache, v_cache, o, lse, BH, l, cap, cache_len, lens, H, pg, scale, st)
                   : prefill_generic_t<__nv_bfloat16, 128>(q, k_cache, v_cache, o, lse, BH, l, cap, cache_len, lens, H, pg, scale,
                                                           st);
}

// pad_to: see cache_append_kernel (1: plain append)
cudaError_t launch_cache_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache, int B, int H,
                                int row_bytes, int l, int cap, int cache_len, const int32_t* lens, const Paging& pg,
                                int pad_to, bool copy_k, cudaStream_t st) {
    const int vec = row_bytes / 16;
    const int64_t n = (int64_t)(l + (pad_to > 1 ? pad_to : 0)) * vec;
    int gx = (int)((n + 255) / 256);
    if (gx > 64) gx = 64;
    if (gx < 1) gx = 1;
    dim3 grid(gx, B * H);
    cache_append_kernel<<<grid, 256, 0, st>>>(static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                                              static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), vec, l, cap, cache_len,
                                              lens, H, pg, pad_to, copy_k ? 1 : 0);
    count_launches(1);
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t prefill_rope_t(const void* q, const void* k_new, void* q_rot, void* k_cache, int BH, int l, int cap,
                                  int cache_len, const int32_t* lens, int H, const Paging& pg, const RopeArgs& rope,
                                  cudaStream_t st) {
    constexpr int RPB = 128 / (D / 2);
    dim3 grid((l + RPB - 1) / RPB, BH);
    prefill_rope_kernel<T, D><<<grid, 128, 0, st>>>(static_cast<const T*>(q), static_cast<const T*>(k_new),
                                                    static_cast<T*>(q_rot), static_cast<T*>(k_cache), l, cap, cache_len, lens,
                                                    H, pg, rope);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_prefill_rope(const void* q, const void* k_new, void* q_rot, void* k_cache, int B, int H, int D, int l,
                                int cap, int cache_len, const int32_t* lens, const Paging& pg, const RopeArgs& rope,
                                loma_dtype dt, cudaStream_t st) {
    const int BH = B * H;
    if (dt == LOMA_F32)
        return D == 64 ? prefill_rope_t<float, 64>(q, k_new, q_rot, k_cache, BH, l, cap, cache_len, lens, H, pg, rope, st)
                       : prefill_rope_t<float, 128>(q, k_new, q_rot, k_cache, BH, l, cap, cache_len, lens, H, pg, rope, st);
    return D == 64 ? prefill_rope_t<__nv_bfloat16, 64>(q, k_new, q_rot, k_cache, BH, l, cap, cache_len, lens, H, pg, rope, st)
                   : prefill_rope_t<__nv_bfloat16, 128>(q, k_new, q_rot, k_cache, BH, l, cap, cache_len, lens, H, pg, rope, st);
}

}  // namespace loma
