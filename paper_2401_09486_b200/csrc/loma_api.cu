// extern "C" boundary of libloma: argument validation and kernel selection.
// Every check happens on the host before anything is enqueued.
#include <limits.h>
#include <math.h>

#include <atomic>

#include "loma_internal.cuh"

namespace loma {

static std::atomic<uint64_t> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
static std::atomic<uint64_t> g_fallbacks{0};

__device__ int g_status_word = 0;

int* device_status_word() {
    // one address per device; looked up on first use with that device current
    static int* addr[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        addr[dev] = static_cast<int*>(p);
    }
    return addr[dev];
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t elt_size(loma_dtype dt) { return dt == LOMA_F32 ? 4 : 2; }

// B200 check, cached per device.  Returns LOMA_OK / LOMA_ERR_UNSUPPORTED / LOMA_ERR_CUDA.
static int check_device() {
    static int cached[64];
    static bool have[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LOMA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return LOMA_ERR_UNSUPPORTED;
    if (!have[dev]) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return LOMA_ERR_CUDA;
        cached[dev] = (major == 10) ? LOMA_OK : LOMA_ERR_UNSUPPORTED;
        have[dev] = true;
    }
    return cached[dev];
}

static int make_layout(int n_chunks, int c, int t, int tail_read, unsigned flags, Layout* L) {
    if (n_chunks < 0 || c < 1 || t < 0 || tail_read < 0) return LOMA_ERR_INVALID_ARG;
    if (t == 0 && n_chunks != 0) return LOMA_ERR_INVALID_ARG;
    const int64_t tc = (int64_t)c * t;
    if (t > 0 && tail_read > tc) return LOMA_ERR_INVALID_ARG;
    const int64_t s = (flags & LOMA_FLAG_NO_REP_ZONE) ? tc + t : 2 * tc + t;
    const int64_t S = (int64_t)n_chunks * s + tail_read;
    if (tc > INT_MAX / 4 || S > INT_MAX) return LOMA_ERR_INVALID_ARG;
    L->n_chunks = n_chunks; L->c = c; L->t = t; L->tc = (int)tc; L->s = (int)s;
    L->tail_read = tail_read; L->S = (int)S; L->flags = flags;
    return LOMA_OK;
}

}  // namespace loma

using namespace loma;

extern "C" {

int loma_version(void) { return 100; }

uint64_t loma_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

uint64_t loma_fallback_count(void) { return g_fallbacks.load(std::memory_order_relaxed); }

const char* loma_status_string(int status) {
    switch (status) {
        case LOMA_OK: return "LOMA_OK";
        case LOMA_ERR_INVALID_ARG: return "LOMA_ERR_INVALID_ARG: invalid argument";
        case LOMA_ERR_UNSUPPORTED: return "LOMA_ERR_UNSUPPORTED: unsupported head dimension, dtype or device";
        case LOMA_ERR_ALIGNMENT: return "LOMA_ERR_ALIGNMENT: pointer or stride not 16-byte aligned";
        case LOMA_ERR_CAPACITY: return "LOMA_ERR_CAPACITY: cache capacity too small";
        case LOMA_ERR_WORKSPACE: return "LOMA_ERR_WORKSPACE: workspace missing or too small";
        case LOMA_ERR_CUDA: return "LOMA_ERR_CUDA: a CUDA call failed";
        case LOMA_ERR_TIMEOUT: return "LOMA_ERR_TIMEOUT: a bounded device-side wait expired";
        default: return "unknown loma status";
    }
}

int loma_layout_index(int n_chunks, int c, int t, int tail_read, unsigned flags, int32_t* chunk, int32_t* zone,
                      int32_t* offset, int32_t* src_token, int32_t* pos_id, int on_device, void* stream) {
    Layout L;
    const int rc = make_layout(n_chunks, c, t, tail_read, flags, &L);
    if (rc != LOMA_OK) return rc;
    if (!on_device) {
        host_layout_index(L, chunk, zone, offset, src_token, pos_id);
        return LOMA_OK;
    }
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    return launch_layout_index(L, chunk, zone, offset, src_token, pos_id, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess
               ? LOMA_OK
               : LOMA_ERR_CUDA;
}

int loma_generation_index(int n_tokens, int c, int t, int32_t* slot, int32_t* pos_id, int32_t* compress_after,
                          int on_device, void* stream) {
    if (n_tokens < 0 || c < 1 || t < 0) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)c * t > INT_MAX / 4) return LOMA_ERR_INVALID_ARG;
    if (!on_device) {
        host_generation_index(n_tokens, c, t, slot, pos_id, compress_after);
        return LOMA_OK;
    }
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    return launch_generation_index(n_tokens, c, t, slot, pos_id, compress_after,
                                   static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? LOMA_OK
               : LOMA_ERR_CUDA;
}

int loma_masked_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int D,
                         int n_chunks, int c, int t, int tc, int tail_read, int64_t stride_b, int64_t stride_h,
                         int64_t stride_s, loma_dtype dtype, float softmax_scale, unsigned flags,
                         void* stream) {
    if (B < 0 || H < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    Layout L;
    const int rc = make_layout(n_chunks, c, t, tail_read, flags, &L);
    if (rc != LOMA_OK) return rc;
    if (tc != L.tc) return LOMA_ERR_INVALID_ARG;
    if (L.S == 0 || B == 0 || H == 0) return LOMA_OK;
    if (!q || !k || !v || !o) return LOMA_ERR_INVALID_ARG;
    if (o == q || o == k || o == v) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (stride_s < D || stride_b < 0 || stride_h < 0) return LOMA_ERR_INVALID_ARG;
    if ((stride_b == 0 && B > 1) || (stride_h == 0 && H > 1)) return LOMA_ERR_INVALID_ARG;   // rows of two (b, h) would coincide
    const size_t es = elt_size(dtype);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return LOMA_ERR_ALIGNMENT;
    if ((stride_b * es) % 16 || (stride_h * es) % 16 || (stride_s * es) % 16) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaErrorNotSupported;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC))
        e = launch_masked_attn_tc(q, k, v, o, lse, B, H, D, L, stride_b, stride_h, stride_s, scale, st);
    if (e == cudaErrorNotSupported) {
        if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC)) g_fallbacks.fetch_add(1, std::memory_order_relaxed);
        e = launch_masked_attn_generic(q, k, v, o, lse, B, H, D, L, stride_b, stride_h, stride_s, dtype, scale, st);
    }
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

size_t loma_masked_attn_bwd_workspace_bytes(int B, int H, int D, int n_chunks, int c, int t, int tail_read,
                                            unsigned flags) {
    (void)D;
    Layout L;
    if (B < 0 || H < 0 || make_layout(n_chunks, c, t, tail_read, flags, &L) != LOMA_OK) return 0;
    const size_t bytes = (size_t)B * H * L.S * sizeof(float);   // delta_i = dO_i . O_i
    return (bytes + 255) & ~(size_t)255;
}

int loma_masked_attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* d_o, const float* lse,
                         void* dq, void* dk, void* dv, int B, int H, int D, int n_chunks, int c, int t, int tc,
                         int tail_read, int64_t stride_b, int64_t stride_h, int64_t stride_s, loma_dtype dtype,
                         float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 0 || H < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    Layout L;
    const int rc = make_layout(n_chunks, c, t, tail_read, flags, &L);
    if (rc != LOMA_OK) return rc;
    if (tc != L.tc) return LOMA_ERR_INVALID_ARG;
    if (L.S == 0 || B == 0 || H == 0) return LOMA_OK;
    const void* ins[5] = {q, k, v, o, d_o};
    void* outs[3] = {dq, dk, dv};
    for (const void* p : ins) if (!p) return LOMA_ERR_INVALID_ARG;
    if (!lse) return LOMA_ERR_INVALID_ARG;
    for (int a = 0; a < 3; ++a) {
        if (!outs[a]) return LOMA_ERR_INVALID_ARG;
        for (const void* p : ins) if (outs[a] == p) return LOMA_ERR_INVALID_ARG;
        for (int b2 = 0; b2 < a; ++b2) if (outs[a] == outs[b2]) return LOMA_ERR_INVALID_ARG;
    }
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (stride_s < D || stride_b < 0 || stride_h < 0) return LOMA_ERR_INVALID_ARG;
    if ((stride_b == 0 && B > 1) || (stride_h == 0 && H > 1)) return LOMA_ERR_INVALID_ARG;   // rows of two (b, h) would coincide
    const size_t es = elt_size(dtype);
    for (const void* p : ins) if (!aligned16(p)) return LOMA_ERR_ALIGNMENT;
    for (void* p : outs) if (!aligned16(p)) return LOMA_ERR_ALIGNMENT;
    if (((uintptr_t)lse & 3u) != 0) return LOMA_ERR_ALIGNMENT;
    if ((stride_b * es) % 16 || (stride_h * es) % 16 || (stride_s * es) % 16) return LOMA_ERR_ALIGNMENT;
    const size_t need = loma_masked_attn_bwd_workspace_bytes(B, H, D, n_chunks, c, t, tail_read, flags);
    if (!workspace || workspace_bytes < need) return LOMA_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* delta = static_cast<float*>(workspace);
    int generic_parts = 3;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC)) {
        const cudaError_t e = launch_masked_attn_bwd_dq_tc(q, k, v, o, d_o, lse, dq, delta, B, H, D, L, stride_b, stride_h,
                                                           stride_s, scale, st);
        if (e == cudaSuccess) {
            generic_parts = 2;
            const cudaError_t e2 = launch_masked_attn_bwd_dkv_tc(q, k, v, d_o, lse, delta, dk, dv, B, H, D, L, stride_b,
                                                                 stride_h, stride_s, scale, st);
            if (e2 == cudaSuccess) return LOMA_OK;
            if (e2 != cudaErrorNotSupported) return LOMA_ERR_CUDA;
        } else if (e != cudaErrorNotSupported) {
            return LOMA_ERR_CUDA;
        }
    }
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC)) g_fallbacks.fetch_add(1, std::memory_order_relaxed);
    const cudaError_t e = launch_masked_attn_bwd_generic(q, k, v, o, d_o, lse, dq, dk, dv, delta, B, H, D, L, stride_b,
                                                         stride_h, stride_s, dtype, scale, generic_parts, st);
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_rope_apply(void* q, void* k, int B, int H, int D, int n_chunks, int c, int t, int tc, int tail_read,
                    int64_t stride_b, int64_t stride_h, int64_t stride_s, loma_dtype dtype, float theta_base,
                    int position_type, unsigned flags, void* stream) {
    if (B < 0 || H < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if (position_type < 0 || position_type > (1 | LOMA_ROPE_INVERSE)) return LOMA_ERR_INVALID_ARG;
    Layout L;
    const int rc = make_layout(n_chunks, c, t, tail_read, flags, &L);
    if (rc != LOMA_OK) return rc;
    if (tc != L.tc) return LOMA_ERR_INVALID_ARG;
    if (L.S == 0 || B == 0 || H == 0 || (!q && !k)) return LOMA_OK;
    if (q && q == k) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (stride_s < D || stride_b < 0 || stride_h < 0) return LOMA_ERR_INVALID_ARG;
    if ((stride_b == 0 && B > 1) || (stride_h == 0 && H > 1)) return LOMA_ERR_INVALID_ARG;   // rows of two (b, h) would coincide
    const size_t es = elt_size(dtype);
    if ((q && !aligned16(q)) || (k && !aligned16(k))) return LOMA_ERR_ALIGNMENT;
    if ((stride_b * es) % 16 || (stride_h * es) % 16 || (stride_s * es) % 16) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const double base = theta_base > 0.f ? (double)theta_base : 10000.0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the kernel skips a NULL tensor
    cudaError_t e = cudaSuccess;
    if (q && k) e = launch_rope(q, k, B, H, D, L, stride_b, stride_h, stride_s, dtype, base, position_type, st);
    else e = launch_rope(q ? q : k, nullptr, B, H, D, L, stride_b, stride_h, stride_s, dtype, base, position_type, st);
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_prefill_cache(const void* k, const void* v, void* k_cache, void* v_cache, int B, int H, int D, int cap,
                       int n_chunks, int c, int t, int tc, int tail_read, int64_t stride_b, int64_t stride_h,
                       int64_t stride_s, loma_dtype dtype, unsigned flags, int* cache_len_out, void* stream) {
    if (B < 0 || H < 0 || cap < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    Layout L;
    const int rc = make_layout(n_chunks, c, t, tail_read, flags, &L);
    if (rc != LOMA_OK) return rc;
    if (tc != L.tc) return LOMA_ERR_INVALID_ARG;
    const int64_t n_rows = (int64_t)n_chunks * t + tail_read;
    if (n_rows > cap) return LOMA_ERR_CAPACITY;
    if (cache_len_out) *cache_len_out = (int)n_rows;
    if (n_rows == 0 || B == 0 || H == 0) return LOMA_OK;
    if (!k || !v || !k_cache || !v_cache) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (stride_s < D || stride_b < 0 || stride_h < 0) return LOMA_ERR_INVALID_ARG;
    if ((stride_b == 0 && B > 1) || (stride_h == 0 && H > 1)) return LOMA_ERR_INVALID_ARG;   // rows of two (b, h) would coincide
    const size_t es = elt_size(dtype);
    if (!aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache)) return LOMA_ERR_ALIGNMENT;
    if ((stride_b * es) % 16 || (stride_h * es) % 16 || (stride_s * es) % 16) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    cudaError_t e = launch_prefill_cache(k, v, k_cache, v_cache, B, H, (int)(D * es), cap, L, stride_b * es, stride_h * es,
                                         stride_s * es, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_masked_attn_plan_coverage(int n_chunks, int c, int t, int tail_read, unsigned flags, uint8_t* counts) {
    Layout L;
    const int rc = make_layout(n_chunks, c, t, tail_read, flags, &L);
    if (rc != LOMA_OK) return rc;
    if (L.S > 0 && !counts) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)L.S * L.S > (1ll << 32)) return LOMA_ERR_INVALID_ARG;
    if (L.S > 0) plan_coverage_host(L, counts);
    return LOMA_OK;
}

int loma_masked_attn_bwd_plan_coverage(int n_chunks, int c, int t, int tail_read, unsigned flags, uint8_t* counts) {
    Layout L;
    const int rc = make_layout(n_chunks, c, t, tail_read, flags, &L);
    if (rc != LOMA_OK) return rc;
    if (L.S > 0 && !counts) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)L.S * L.S > (1ll << 32)) return LOMA_ERR_INVALID_ARG;
    if (L.S > 0) plan_coverage_by_key_host(L, counts);
    return LOMA_OK;
}

size_t loma_decode_workspace_bytes(int B, int H, int D, int cache_len) {
    if (B <= 0 || H <= 0 || D <= 0 || cache_len < 0) return 0;
    return decode_workspace_bytes(B * H, D, cache_len + 1);
}

static int decode_attn_impl(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                            float* lse, int B, int H, int D, int cap, int cache_len, loma_dtype dtype,
                            float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes,
                            void* stream, const RopeArgs& rope) {
    if (B < 0 || H < 0 || cap < 0 || cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((k_new == nullptr) != (v_new == nullptr)) return LOMA_ERR_INVALID_ARG;
    if (cache_len >= cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0) return LOMA_OK;
    if (!q || !k_cache || !v_cache || !o) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new) || !aligned16(workspace))
        return LOMA_ERR_ALIGNMENT;
    const size_t need = loma_decode_workspace_bytes(B, H, D, cache_len);
    if (need > 0 && (!workspace || workspace_bytes < need)) return LOMA_ERR_WORKSPACE;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((int64_t)B * H * 128 > INT_MAX) return LOMA_ERR_INVALID_ARG;
    cudaError_t e;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC))
        e = launch_decode_bf16(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_len, nullptr, scale,
                               workspace, Paging{}, st, rope);
    else
        e = launch_decode_generic(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_len, nullptr, dtype,
                                  scale, Paging{}, st, rope);
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_decode_attn(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                     float* lse, int B, int H, int D, int cap, int cache_len, loma_dtype dtype,
                     float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes,
                     void* stream) {
    return decode_attn_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_len, dtype, softmax_scale, flags,
                            workspace, workspace_bytes, stream, RopeArgs{});
}

int loma_decode_attn_rope(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                          float* lse, int B, int H, int D, int cap, int cache_len, int pos, float theta_base,
                          loma_dtype dtype, float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes,
                          void* stream) {
    if (pos < 0) return LOMA_ERR_INVALID_ARG;
    if (B > 0 && H > 0 && (!k_new || !v_new)) return LOMA_ERR_INVALID_ARG;   // the key to rotate has to be given
    RopeArgs rope;
    rope.on = 1; rope.pos0 = pos; rope.stride = 0;
    rope.log2_base = log2(theta_base > 0.f ? (double)theta_base : 10000.0);
    return decode_attn_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_len, dtype, softmax_scale, flags,
                            workspace, workspace_bytes, stream, rope);
}

// ---- the generator's loop over layers (Appendix A: `for i in range(len(self.kv_cache))`) ------------------
int loma_decode_attn_layers(int n_layers, const void* const* q, const void* const* k_new, const void* const* v_new,
                            void* const* k_cache, void* const* v_cache, void* const* o, float* const* lse, int B, int H,
                            int D, int cap, int cache_len, loma_dtype dtype, float softmax_scale, unsigned flags,
                            void* workspace, size_t workspace_bytes, void* stream) {
    if (n_layers < 0) return LOMA_ERR_INVALID_ARG;
    if (n_layers > 0 && (!q || !k_cache || !v_cache || !o)) return LOMA_ERR_INVALID_ARG;
    // every layer is validated before the first one is enqueued (nothing runs on an error)
    for (int pass = 0; pass < 2; ++pass) {
        for (int i = 0; i < n_layers; ++i) {
            const void* kn = k_new ? k_new[i] : nullptr;
            const void* vn = v_new ? v_new[i] : nullptr;
            float* ls = lse ? lse[i] : nullptr;
            if (pass == 0) {
                if ((kn == nullptr) != (vn == nullptr)) return LOMA_ERR_INVALID_ARG;
                if (B > 0 && H > 0 && (!q[i] || !k_cache[i] || !v_cache[i] || !o[i])) return LOMA_ERR_INVALID_ARG;
                if (!aligned16(q[i]) || !aligned16(k_cache[i]) || !aligned16(v_cache[i]) || !aligned16(o[i]) || !aligned16(kn) ||
                    !aligned16(vn))
                    return LOMA_ERR_ALIGNMENT;
                for (int j = 0; j < i; ++j)
                    if (k_cache[j] == k_cache[i] || v_cache[j] == v_cache[i] || o[j] == o[i]) return LOMA_ERR_INVALID_ARG;
            } else {
                // the layers share the workspace: they run one after the other on the stream
                const int rc = loma_decode_attn(q[i], kn, vn, k_cache[i], v_cache[i], o[i], ls, B, H, D, cap, cache_len, dtype,
                                                softmax_scale, flags, workspace, workspace_bytes, stream);
                if (rc != LOMA_OK) return rc;
            }
        }
        if (pass == 0 && n_layers > 0) {
            // the scalar arguments: checked once through a call that launches nothing (B = 0 is a no-op after validation)
            if (B < 0 || H < 0 || cap < 0 || cache_len < 0) return LOMA_ERR_INVALID_ARG;
            if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
            if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
            if (cache_len >= cap) return LOMA_ERR_CAPACITY;
            if (!aligned16(workspace)) return LOMA_ERR_ALIGNMENT;
            const size_t need = loma_decode_workspace_bytes(B, H, D, cache_len);
            if (B > 0 && H > 0 && need > 0 && (!workspace || workspace_bytes < need)) return LOMA_ERR_WORKSPACE;
        }
    }
    return LOMA_OK;
}

int loma_compress_step_layers(int n_layers, const void* const* q_mem, const void* const* k_mem, const void* const* v_mem,
                              void* const* k_cache, void* const* v_cache, void* const* o_mem, float* const* lse, int B,
                              int H, int D, int cap, int mem_len, int c, int t, int tc, loma_dtype dtype,
                              float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, void* stream) {
    if (n_layers < 0) return LOMA_ERR_INVALID_ARG;
    if (n_layers > 0 && (!q_mem || !k_mem || !v_mem || !k_cache || !v_cache || !o_mem)) return LOMA_ERR_INVALID_ARG;
    if (n_layers > 0) {
        if (B < 0 || H < 0 || cap < 0 || mem_len < 0 || c < 1 || t < 1) return LOMA_ERR_INVALID_ARG;
        if ((int64_t)c * t != (int64_t)tc) return LOMA_ERR_INVALID_ARG;
        if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
        if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
        if ((int64_t)mem_len + tc > (int64_t)cap) return LOMA_ERR_CAPACITY;
        if (!aligned16(workspace)) return LOMA_ERR_ALIGNMENT;
        const size_t need = loma_compress_workspace_bytes(B, H, D, t, mem_len, flags);
        if (B > 0 && H > 0 && need > 0 && (!workspace || workspace_bytes < need)) return LOMA_ERR_WORKSPACE;
    }
    for (int i = 0; i < n_layers; ++i) {
        if (B > 0 && H > 0 && (!q_mem[i] || !k_mem[i] || !v_mem[i] || !k_cache[i] || !v_cache[i] || !o_mem[i]))
            return LOMA_ERR_INVALID_ARG;
        if (!aligned16(q_mem[i]) || !aligned16(k_mem[i]) || !aligned16(v_mem[i]) || !aligned16(k_cache[i]) ||
            !aligned16(v_cache[i]) || !aligned16(o_mem[i]))
            return LOMA_ERR_ALIGNMENT;
        for (int j = 0; j < i; ++j)
            if (k_cache[j] == k_cache[i] || v_cache[j] == v_cache[i] || o_mem[j] == o_mem[i]) return LOMA_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n_layers; ++i) {
        const int rc = loma_compress_step(q_mem[i], k_mem[i], v_mem[i], k_cache[i], v_cache[i], o_mem[i], lse ? lse[i] : nullptr,
                                          B, H, D, cap, mem_len, c, t, tc, dtype, softmax_scale, flags, workspace,
                                          workspace_bytes, stream);
        if (rc != LOMA_OK) return rc;
    }
    return LOMA_OK;
}

static int log2_exact(int x);   // defined with the paged entry points below

// The three forms of the prompt piece over a cache.  cache_len: the uniform length, or (cache_lens given) the bound the
// per-sequence lengths are clamped to; pg.table given: the cache is the paged pool and cap = max_pages * page_size.
static int prefill_attn_impl(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                             float* lse, int B, int H, int D, int l, int cap, int cache_len, const int32_t* cache_lens,
                             const Paging& pg, loma_dtype dtype, float softmax_scale, unsigned flags, void* stream,
                             const RopeArgs& rope = RopeArgs{}) {
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the tensor-core kernel (bf16; a handful of rows is cheaper on CUDA cores, one warp per row:
    // from 8 rows on one pass of the cache through the tensor-core kernel wins over l passes)
    // (over a paged cache only when a page holds a multiple of 128 rows: a 128-key tile then lies in one page)
    const bool tc = dtype == LOMA_BF16 && l >= 8 && (!pg.table || pg.log2_ps >= 7) && !(flags & LOMA_FLAG_FORCE_GENERIC);
    // 1. the new tokens' K/V go into the cache (bit-exact); 2. every new row attends to cache rows 0 .. len + i.
    // With per-sequence lengths the tensor-core kernel also wants the rest of each sequence's last 128-row key tile finite.
    const int pad_to = (tc && cache_lens) ? 128 : 1;
    if (k_new || pad_to > 1) {
        if (launch_cache_append(k_new, v_new, k_cache, v_cache, B, H, (int)(D * elt_size(dtype)), l, cap, cache_len,
                                cache_lens, pg, pad_to, !rope.on, st) != cudaSuccess)
            return LOMA_ERR_CUDA;
    }
    if (rope.on) {
        // Section 4.5: q and the new keys are rotated at the ids cursor + i.  The rotated keys go straight into the
        // cache; the rotated queries into o, which the attention kernels below then read as their query (every
        // tile or row reads its own query rows before it writes the same rows of the output).
        if (launch_prefill_rope(q, k_new, o, k_cache, B, H, D, l, cap, cache_len, cache_lens, pg, rope, dtype, st) !=
            cudaSuccess)
            return LOMA_ERR_CUDA;
        q = o;
    }
    cudaError_t e = cudaErrorNotSupported;
    if (tc) {
        e = launch_prefill_attn_tc(q, k_cache, v_cache, o, lse, B, H, D, l, cap, cache_len, cache_lens, pg, scale, st);
        if (e == cudaErrorNotSupported) g_fallbacks.fetch_add(1, std::memory_order_relaxed);
    }
    if (e == cudaErrorNotSupported)
        e = launch_prefill_attn_generic(q, k_cache, v_cache, o, lse, B, H, D, l, cap, cache_len, cache_lens, pg, dtype,
                                        scale, st);
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_prefill_attn(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                      float* lse, int B, int H, int D, int l, int cap, int cache_len, loma_dtype dtype,
                      float softmax_scale, unsigned flags, void* stream) {
    if (B < 0 || H < 0 || l < 0 || cap < 0 || cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((k_new == nullptr) != (v_new == nullptr)) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)cache_len + l > cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0 || l == 0) return LOMA_OK;
    if (!q || !k_cache || !v_cache || !o) return LOMA_ERR_INVALID_ARG;
    if (o == q || o == k_new || o == v_new) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new))
        return LOMA_ERR_ALIGNMENT;
    if (lse && ((uintptr_t)lse & 3u)) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    return prefill_attn_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, l, cap, cache_len, nullptr, Paging{}, dtype,
                             softmax_scale, flags, stream);
}

int loma_prefill_attn_ragged(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                             float* lse, int B, int H, int D, int l, int cap, const int32_t* cache_lens,
                             int max_cache_len, loma_dtype dtype, float softmax_scale, unsigned flags, void* stream) {
    if (B < 0 || H < 0 || l < 0 || cap < 0 || max_cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((k_new == nullptr) != (v_new == nullptr)) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)max_cache_len + l > cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0 || l == 0) return LOMA_OK;
    if (!q || !k_cache || !v_cache || !o || !cache_lens) return LOMA_ERR_INVALID_ARG;
    if (o == q || o == k_new || o == v_new) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new) || ((uintptr_t)cache_lens & 3u))
        return LOMA_ERR_ALIGNMENT;
    if (lse && ((uintptr_t)lse & 3u)) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    return prefill_attn_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, l, cap, max_cache_len, cache_lens, Paging{},
                             dtype, softmax_scale, flags, stream);
}

int loma_prefill_attn_paged(const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                            const int32_t* block_table, void* o, float* lse, int B, int H, int D, int l, int page_size,
                            int max_pages, int n_pages, const int32_t* cache_lens, int max_cache_len, loma_dtype dtype,
                            float softmax_scale, unsigned flags, void* stream) {
    if (B < 0 || H < 0 || l < 0 || max_pages < 0 || n_pages < 0 || max_cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    const int l2 = log2_exact(page_size);
    if (l2 < 0 || page_size > 65536) return LOMA_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr)) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)max_cache_len + l > (int64_t)max_pages * page_size) return LOMA_ERR_CAPACITY;
    if ((int64_t)max_pages * page_size > INT_MAX) return LOMA_ERR_INVALID_ARG;
    if (B == 0 || H == 0 || l == 0) return LOMA_OK;
    if (!q || !k_pool || !v_pool || !o || !block_table || !cache_lens || n_pages < 1) return LOMA_ERR_INVALID_ARG;
    if (o == q || o == k_new || o == v_new) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_pool) || !aligned16(v_pool) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new) || ((uintptr_t)cache_lens & 3u) || ((uintptr_t)block_table & 3u))
        return LOMA_ERR_ALIGNMENT;
    if (lse && ((uintptr_t)lse & 3u)) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    Paging pg;
    pg.table = block_table; pg.max_pages = max_pages; pg.log2_ps = l2; pg.n_pages = n_pages;
    return prefill_attn_impl(q, k_new, v_new, k_pool, v_pool, o, lse, B, H, D, l, max_pages * page_size, max_cache_len,
                             cache_lens, pg, dtype, softmax_scale, flags, stream);
}

// The prompt piece with the rotation fused in.  Shared checks of the three forms; then the plain entry point's own.
static int prefill_rope_args(int B, int H, int l, const void* k_new, const void* v_new, int pos0, const int32_t* positions,
                             bool per_sequence, float theta_base, RopeArgs* rope) {
    if (B > 0 && H > 0 && l > 0 && (!k_new || !v_new)) return LOMA_ERR_INVALID_ARG;   // the keys to rotate have to be given
    if (per_sequence) {
        if (B > 0 && H > 0 && l > 0 && !positions) return LOMA_ERR_INVALID_ARG;
        if ((uintptr_t)positions & 3u) return LOMA_ERR_ALIGNMENT;
    } else if (pos0 < 0 || (l > 0 && (int64_t)pos0 + l - 1 > INT_MAX)) {
        return LOMA_ERR_INVALID_ARG;
    }
    rope->on = 1; rope->pos0 = pos0; rope->stride = 1; rope->pos_seq = per_sequence ? positions : nullptr;
    rope->log2_base = log2(theta_base > 0.f ? (double)theta_base : 10000.0);
    return LOMA_OK;
}

int loma_prefill_attn_rope(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                           float* lse, int B, int H, int D, int l, int cap, int cache_len, int pos0, float theta_base,
                           loma_dtype dtype, float softmax_scale, unsigned flags, void* stream) {
    RopeArgs rope;
    const int rc = prefill_rope_args(B, H, l, k_new, v_new, pos0, nullptr, false, theta_base, &rope);
    if (rc != LOMA_OK) return rc;
    if (B < 0 || H < 0 || l < 0 || cap < 0 || cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((int64_t)cache_len + l > cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0 || l == 0) return LOMA_OK;
    if (!q || !k_cache || !v_cache || !o) return LOMA_ERR_INVALID_ARG;
    if (o == q || o == k_new || o == v_new) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new))
        return LOMA_ERR_ALIGNMENT;
    if (lse && ((uintptr_t)lse & 3u)) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    return prefill_attn_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, l, cap, cache_len, nullptr, Paging{}, dtype,
                             softmax_scale, flags, stream, rope);
}

int loma_prefill_attn_ragged_rope(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                  void* o, float* lse, int B, int H, int D, int l, int cap, const int32_t* cache_lens,
                                  int max_cache_len, const int32_t* positions, float theta_base, loma_dtype dtype,
                                  float softmax_scale, unsigned flags, void* stream) {
    RopeArgs rope;
    const int rc = prefill_rope_args(B, H, l, k_new, v_new, 0, positions, true, theta_base, &rope);
    if (rc != LOMA_OK) return rc;
    if (B < 0 || H < 0 || l < 0 || cap < 0 || max_cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((int64_t)max_cache_len + l > cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0 || l == 0) return LOMA_OK;
    if (!q || !k_cache || !v_cache || !o || !cache_lens) return LOMA_ERR_INVALID_ARG;
    if (o == q || o == k_new || o == v_new) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new) || ((uintptr_t)cache_lens & 3u))
        return LOMA_ERR_ALIGNMENT;
    if (lse && ((uintptr_t)lse & 3u)) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    return prefill_attn_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, l, cap, max_cache_len, cache_lens, Paging{},
                             dtype, softmax_scale, flags, stream, rope);
}

int loma_prefill_attn_paged_rope(const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                                 const int32_t* block_table, void* o, float* lse, int B, int H, int D, int l,
                                 int page_size, int max_pages, int n_pages, const int32_t* cache_lens, int max_cache_len,
                                 const int32_t* positions, float theta_base, loma_dtype dtype, float softmax_scale,
                                 unsigned flags, void* stream) {
    RopeArgs rope;
    const int rc = prefill_rope_args(B, H, l, k_new, v_new, 0, positions, true, theta_base, &rope);
    if (rc != LOMA_OK) return rc;
    if (B < 0 || H < 0 || l < 0 || max_pages < 0 || n_pages < 0 || max_cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    const int l2 = log2_exact(page_size);
    if (l2 < 0 || page_size > 65536) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)max_cache_len + l > (int64_t)max_pages * page_size) return LOMA_ERR_CAPACITY;
    if ((int64_t)max_pages * page_size > INT_MAX) return LOMA_ERR_INVALID_ARG;
    if (B == 0 || H == 0 || l == 0) return LOMA_OK;
    if (!q || !k_pool || !v_pool || !o || !block_table || !cache_lens || n_pages < 1) return LOMA_ERR_INVALID_ARG;
    if (o == q || o == k_new || o == v_new) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)B * H > 65535) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_pool) || !aligned16(v_pool) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new) || ((uintptr_t)cache_lens & 3u) || ((uintptr_t)block_table & 3u))
        return LOMA_ERR_ALIGNMENT;
    if (lse && ((uintptr_t)lse & 3u)) return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    Paging pg;
    pg.table = block_table; pg.max_pages = max_pages; pg.log2_ps = l2; pg.n_pages = n_pages;
    return prefill_attn_impl(q, k_new, v_new, k_pool, v_pool, o, lse, B, H, D, l, max_pages * page_size, max_cache_len,
                             cache_lens, pg, dtype, softmax_scale, flags, stream, rope);
}

int loma_prefill_attn_plan_coverage(int l, int cache_len, uint8_t* counts) {
    if (l < 0 || cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)l * ((int64_t)l + cache_len) > (1ll << 32)) return LOMA_ERR_INVALID_ARG;
    if (l > 0 && !counts) return LOMA_ERR_INVALID_ARG;
    if (l > 0) prefill_plan_coverage_host(l, cache_len, counts);
    return LOMA_OK;
}

static int loma_decode_attn_ragged_impl(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                        void* v_cache, void* o,
                            float* lse, int B, int H, int D, int cap, const int32_t* cache_lens, int max_cache_len,
                            loma_dtype dtype, float softmax_scale, unsigned flags, void* workspace,
                            size_t workspace_bytes, void* stream, const RopeArgs& rope) {
    if (B < 0 || H < 0 || cap < 0 || max_cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((k_new == nullptr) != (v_new == nullptr)) return LOMA_ERR_INVALID_ARG;
    if (max_cache_len >= cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0) return LOMA_OK;
    if (!q || !k_cache || !v_cache || !o || !cache_lens) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new) || !aligned16(workspace) || ((uintptr_t)cache_lens & 3u))
        return LOMA_ERR_ALIGNMENT;
    const size_t need = loma_decode_workspace_bytes(B, H, D, max_cache_len);
    if (need > 0 && (!workspace || workspace_bytes < need)) return LOMA_ERR_WORKSPACE;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((int64_t)B * H * 128 > INT_MAX) return LOMA_ERR_INVALID_ARG;
    cudaError_t e;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC))
        e = launch_decode_bf16(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, max_cache_len, cache_lens, scale,
                               workspace, Paging{}, st, rope);
    else
        e = launch_decode_generic(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, max_cache_len, cache_lens,
                                  dtype, scale, Paging{}, st, rope);
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_decode_attn_ragged(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache, void* o,
                            float* lse, int B, int H, int D, int cap, const int32_t* cache_lens, int max_cache_len,
                            loma_dtype dtype, float softmax_scale, unsigned flags, void* workspace,
                            size_t workspace_bytes, void* stream) {
    return loma_decode_attn_ragged_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_lens,
                                        max_cache_len, dtype, softmax_scale, flags, workspace, workspace_bytes,
                                        stream, RopeArgs{});
}

int loma_decode_attn_ragged_rope(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                 void* o, float* lse, int B, int H, int D, int cap, const int32_t* cache_lens,
                                 int max_cache_len, const int32_t* positions, float theta_base, loma_dtype dtype,
                                 float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes,
                                 void* stream) {
    if (B > 0 && H > 0 && (!positions || !k_new || !v_new)) return LOMA_ERR_INVALID_ARG;
    if ((uintptr_t)positions & 3u) return LOMA_ERR_ALIGNMENT;
    RopeArgs rope;
    rope.on = 1; rope.pos_seq = positions; rope.stride = 0;
    rope.log2_base = log2(theta_base > 0.f ? (double)theta_base : 10000.0);
    return loma_decode_attn_ragged_impl(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_lens,
                                        max_cache_len, dtype, softmax_scale, flags, workspace, workspace_bytes,
                                        stream, rope);
}

// page_size must be a power of two; returns its log2 or -1
static int log2_exact(int x) {
    if (x <= 0 || (x & (x - 1))) return -1;
    int l = 0;
    while ((1 << l) < x) ++l;
    return l;
}

static int loma_decode_attn_paged_impl(const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                           const int32_t* block_table, void* o, float* lse, int B, int H, int D, int page_size,
                           int max_pages, int n_pages, const int32_t* cache_lens, int max_cache_len, loma_dtype dtype,
                           float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, void* stream,
                                   const RopeArgs& rope) {
    if (B < 0 || H < 0 || max_pages < 0 || n_pages < 0 || max_cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    const int l2 = log2_exact(page_size);
    if (l2 < 0 || page_size > 65536) return LOMA_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr)) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)max_cache_len >= (int64_t)max_pages * page_size) return LOMA_ERR_CAPACITY;   // the new token needs a slot too
    if (B == 0 || H == 0) return LOMA_OK;
    if (!q || !k_pool || !v_pool || !o || !block_table || !cache_lens || n_pages < 1) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_pool) || !aligned16(v_pool) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new) || !aligned16(workspace) || ((uintptr_t)cache_lens & 3u) || ((uintptr_t)block_table & 3u))
        return LOMA_ERR_ALIGNMENT;
    const size_t need = loma_decode_workspace_bytes(B, H, D, max_cache_len);
    if (need > 0 && (!workspace || workspace_bytes < need)) return LOMA_ERR_WORKSPACE;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((int64_t)B * H * 128 > INT_MAX) return LOMA_ERR_INVALID_ARG;
    Paging pg;
    pg.table = block_table; pg.max_pages = max_pages; pg.log2_ps = l2; pg.n_pages = n_pages;
    cudaError_t e;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC))
        e = launch_decode_bf16(q, k_new, v_new, k_pool, v_pool, o, lse, B, H, D, 0, max_cache_len, cache_lens, scale,
                               workspace, pg, st, rope);
    else
        e = launch_decode_generic(q, k_new, v_new, k_pool, v_pool, o, lse, B, H, D, 0, max_cache_len, cache_lens, dtype,
                                  scale, pg, st, rope);
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_decode_attn_paged(const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                           const int32_t* block_table, void* o, float* lse, int B, int H, int D, int page_size,
                           int max_pages, int n_pages, const int32_t* cache_lens, int max_cache_len, loma_dtype dtype,
                           float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes, void* stream) {
    return loma_decode_attn_paged_impl(q, k_new, v_new, k_pool, v_pool, block_table, o, lse, B, H, D, page_size,
                                       max_pages, n_pages, cache_lens, max_cache_len, dtype, softmax_scale, flags,
                                       workspace, workspace_bytes, stream, RopeArgs{});
}

int loma_decode_attn_paged_rope(const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                                const int32_t* block_table, void* o, float* lse, int B, int H, int D, int page_size,
                                int max_pages, int n_pages, const int32_t* cache_lens, int max_cache_len,
                                const int32_t* positions, float theta_base, loma_dtype dtype, float softmax_scale,
                                unsigned flags, void* workspace, size_t workspace_bytes, void* stream) {
    if (B > 0 && H > 0 && (!positions || !k_new || !v_new)) return LOMA_ERR_INVALID_ARG;
    if ((uintptr_t)positions & 3u) return LOMA_ERR_ALIGNMENT;
    RopeArgs rope;
    rope.on = 1; rope.pos_seq = positions; rope.stride = 0;
    rope.log2_base = log2(theta_base > 0.f ? (double)theta_base : 10000.0);
    return loma_decode_attn_paged_impl(q, k_new, v_new, k_pool, v_pool, block_table, o, lse, B, H, D, page_size,
                                       max_pages, n_pages, cache_lens, max_cache_len, dtype, softmax_scale, flags,
                                       workspace, workspace_bytes, stream, rope);
}

static int loma_compress_step_paged_impl(const void* q_mem, const void* k_mem, const void* v_mem, void* k_pool, void* v_pool,
                             const int32_t* block_table, void* o_mem, float* lse, int B, int H, int D, int page_size,
                             int max_pages, int n_pages, const int32_t* mem_lens, int max_mem_len, int c, int t, int tc,
                             loma_dtype dtype, float softmax_scale, unsigned flags, void* stream, const RopeArgs& rope) {
    if (B < 0 || H < 0 || max_pages < 0 || n_pages < 0 || max_mem_len < 0 || c < 1 || t < 1) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)c * t != (int64_t)tc) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if (flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM) return LOMA_ERR_UNSUPPORTED;
    const int l2 = log2_exact(page_size);
    if (l2 < 0 || page_size > 65536) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)max_mem_len + tc > (int64_t)max_pages * page_size) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0) return LOMA_OK;
    if (!q_mem || !k_mem || !v_mem || !k_pool || !v_pool || !o_mem || !mem_lens || !block_table || n_pages < 1)
        return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q_mem) || !aligned16(k_mem) || !aligned16(v_mem) || !aligned16(k_pool) || !aligned16(v_pool) ||
        !aligned16(o_mem) || ((uintptr_t)mem_lens & 3u) || ((uintptr_t)block_table & 3u))
        return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((int64_t)B * H * 256 > INT_MAX) return LOMA_ERR_INVALID_ARG;
    Paging pg;
    pg.table = block_table; pg.max_pages = max_pages; pg.log2_ps = l2; pg.n_pages = n_pages;
    cudaError_t e;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC) && t <= (rope.on ? 16 : 128))
        e = launch_compress_bf16(q_mem, k_mem, v_mem, k_pool, v_pool, o_mem, lse, B, H, D, 0, max_mem_len, mem_lens, c, t, flags,
                                 scale, nullptr, pg, st, rope);
    else
        e = launch_compress_generic(q_mem, k_mem, v_mem, k_pool, v_pool, o_mem, lse, B, H, D, 0, max_mem_len, mem_lens, c, t,
                                    dtype, scale, flags, pg, st, rope);
    if (e == cudaErrorNotSupported) return LOMA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_compress_step_paged(const void* q_mem, const void* k_mem, const void* v_mem, void* k_pool, void* v_pool,
                             const int32_t* block_table, void* o_mem, float* lse, int B, int H, int D, int page_size,
                             int max_pages, int n_pages, const int32_t* mem_lens, int max_mem_len, int c, int t, int tc,
                             loma_dtype dtype, float softmax_scale, unsigned flags, void* stream) {
    return loma_compress_step_paged_impl(q_mem, k_mem, v_mem, k_pool, v_pool, block_table, o_mem, lse, B, H, D,
                                         page_size, max_pages, n_pages, mem_lens, max_mem_len, c, t, tc, dtype,
                                         softmax_scale, flags, stream, RopeArgs{});
}

int loma_compress_step_paged_rope(const void* q_mem, const void* k_mem, const void* v_mem, void* k_pool, void* v_pool,
                                  const int32_t* block_table, void* o_mem, float* lse, int B, int H, int D,
                                  int page_size, int max_pages, int n_pages, const int32_t* mem_lens, int max_mem_len,
                                  int c, int t, int tc, const int32_t* pos0s, int pos_stride, float theta_base,
                                  loma_dtype dtype, float softmax_scale, unsigned flags, void* stream) {
    if (pos_stride < 0) return LOMA_ERR_INVALID_ARG;
    if (B > 0 && H > 0 && !pos0s) return LOMA_ERR_INVALID_ARG;
    if ((uintptr_t)pos0s & 3u) return LOMA_ERR_ALIGNMENT;
    RopeArgs rope;
    rope.on = 1; rope.pos_seq = pos0s; rope.stride = pos_stride;
    rope.log2_base = log2(theta_base > 0.f ? (double)theta_base : 10000.0);
    return loma_compress_step_paged_impl(q_mem, k_mem, v_mem, k_pool, v_pool, block_table, o_mem, lse, B, H, D,
                                         page_size, max_pages, n_pages, mem_lens, max_mem_len, c, t, tc, dtype,
                                         softmax_scale, flags, stream, rope);
}

size_t loma_decode_static_scratch_bytes(void) { return decode_static_scratch_bytes(); }

int loma_decode_attn_static(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                            void* o, float* lse, int B, int H, int D, int cap, int cache_len, loma_dtype dtype,
                            float softmax_scale, void* stream) {
    if (B < 0 || H < 0 || cap < 0 || cache_len < 0) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((k_new == nullptr) != (v_new == nullptr)) return LOMA_ERR_INVALID_ARG;
    if (cache_len >= cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0) return LOMA_OK;
    if (!q || !k_cache || !v_cache || !o) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(k_new) ||
        !aligned16(v_new))
        return LOMA_ERR_ALIGNMENT;
    if ((int64_t)B * H * 128 > INT_MAX) return LOMA_ERR_INVALID_ARG;
    // the request must fit the built-in scratch array
    if (decode_workspace_bytes(B * H, D, cache_len + 1) > decode_static_scratch_bytes()) return LOMA_ERR_WORKSPACE;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaError_t e = launch_decode_bf16_static(q, k_new, v_new, k_cache, v_cache, o, lse, B, H, D, cap, cache_len,
                                              scale, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

size_t loma_compress_workspace_bytes(int B, int H, int D, int t, int mem_len, unsigned flags) {
    if (B <= 0 || H <= 0 || D <= 0 || t <= 0 || mem_len < 0) return 0;
    return compress_workspace_bytes(B * H, D, t, mem_len, flags);
}

static int compress_step_impl(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache, void* v_cache,
                              void* o_mem, float* lse, int B, int H, int D, int cap, int mem_len, int c, int t, int tc,
                              loma_dtype dtype, float softmax_scale, unsigned flags, void* workspace,
                              size_t workspace_bytes, void* stream, const RopeArgs& rope) {
    if (B < 0 || H < 0 || cap < 0 || mem_len < 0 || c < 1 || t < 1) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)c * t != (int64_t)tc) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if ((int64_t)mem_len + tc > (int64_t)cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0) return LOMA_OK;
    if (!q_mem || !k_mem || !v_mem || !k_cache || !v_cache || !o_mem) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q_mem) || !aligned16(k_mem) || !aligned16(v_mem) || !aligned16(k_cache) ||
        !aligned16(v_cache) || !aligned16(o_mem) || !aligned16(workspace))
        return LOMA_ERR_ALIGNMENT;
    const size_t need = loma_compress_workspace_bytes(B, H, D, t, mem_len, flags);
    if (need > 0 && (!workspace || workspace_bytes < need)) return LOMA_ERR_WORKSPACE;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((int64_t)B * H * 256 > INT_MAX) return LOMA_ERR_INVALID_ARG;
    cudaError_t e = cudaErrorNotSupported;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC) && t <= (rope.on ? 16 : 128))
        e = launch_compress_bf16(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, mem_len, nullptr, c, t,
                                 flags, scale, workspace, Paging{}, st, rope);
    if (e == cudaErrorNotSupported)
        e = launch_compress_generic(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, mem_len, nullptr, c,
                                    t, dtype, scale, flags, Paging{}, st, rope);
    if (e == cudaErrorNotSupported) return LOMA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_compress_step(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache, void* v_cache,
                       void* o_mem, float* lse, int B, int H, int D, int cap, int mem_len, int c, int t, int tc,
                       loma_dtype dtype, float softmax_scale, unsigned flags, void* workspace,
                       size_t workspace_bytes, void* stream) {
    return compress_step_impl(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, mem_len, c, t, tc, dtype,
                              softmax_scale, flags, workspace, workspace_bytes, stream, RopeArgs{});
}

int loma_compress_step_rope(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache, void* v_cache,
                            void* o_mem, float* lse, int B, int H, int D, int cap, int mem_len, int c, int t, int tc,
                            int pos0, int pos_stride, float theta_base, loma_dtype dtype, float softmax_scale,
                            unsigned flags, void* workspace, size_t workspace_bytes, void* stream) {
    if (pos0 < 0 || pos_stride < 0) return LOMA_ERR_INVALID_ARG;
    if (t > 0 && (int64_t)pos0 + (int64_t)(t - 1) * pos_stride > INT_MAX) return LOMA_ERR_INVALID_ARG;
    RopeArgs rope;
    rope.on = 1; rope.pos0 = pos0; rope.stride = pos_stride;
    rope.log2_base = log2(theta_base > 0.f ? (double)theta_base : 10000.0);
    return compress_step_impl(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, mem_len, c, t, tc, dtype,
                              softmax_scale, flags, workspace, workspace_bytes, stream, rope);
}

static int loma_compress_step_ragged_impl(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache, void* v_cache,
                              void* o_mem, float* lse, int B, int H, int D, int cap, const int32_t* mem_lens,
                              int max_mem_len, int c, int t, int tc, loma_dtype dtype, float softmax_scale, unsigned flags,
                              void* stream, const RopeArgs& rope) {
    if (B < 0 || H < 0 || cap < 0 || max_mem_len < 0 || c < 1 || t < 1) return LOMA_ERR_INVALID_ARG;
    if ((int64_t)c * t != (int64_t)tc) return LOMA_ERR_INVALID_ARG;
    if (dtype != LOMA_F32 && dtype != LOMA_BF16) return LOMA_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return LOMA_ERR_UNSUPPORTED;
    if (flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM) return LOMA_ERR_UNSUPPORTED;   // the split of earlier memory is sized per call
    if ((int64_t)max_mem_len + tc > (int64_t)cap) return LOMA_ERR_CAPACITY;
    if (B == 0 || H == 0) return LOMA_OK;
    if (!q_mem || !k_mem || !v_mem || !k_cache || !v_cache || !o_mem || !mem_lens) return LOMA_ERR_INVALID_ARG;
    if (!aligned16(q_mem) || !aligned16(k_mem) || !aligned16(v_mem) || !aligned16(k_cache) || !aligned16(v_cache) ||
        !aligned16(o_mem) || ((uintptr_t)mem_lens & 3u))
        return LOMA_ERR_ALIGNMENT;
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((int64_t)B * H * 256 > INT_MAX) return LOMA_ERR_INVALID_ARG;
    cudaError_t e;
    if (dtype == LOMA_BF16 && !(flags & LOMA_FLAG_FORCE_GENERIC) && t <= (rope.on ? 16 : 128))
        e = launch_compress_bf16(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, max_mem_len, mem_lens, c, t,
                                 flags, scale, nullptr, Paging{}, st, rope);
    else
        e = launch_compress_generic(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, max_mem_len, mem_lens,
                                    c, t, dtype, scale, flags, Paging{}, st, rope);
    return e == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_compress_step_ragged(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache, void* v_cache,
                              void* o_mem, float* lse, int B, int H, int D, int cap, const int32_t* mem_lens,
                              int max_mem_len, int c, int t, int tc, loma_dtype dtype, float softmax_scale, unsigned flags,
                              void* stream) {
    return loma_compress_step_ragged_impl(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, mem_lens,
                                          max_mem_len, c, t, tc, dtype, softmax_scale, flags, stream, RopeArgs{});
}

int loma_compress_step_ragged_rope(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache,
                                   void* v_cache, void* o_mem, float* lse, int B, int H, int D, int cap,
                                   const int32_t* mem_lens, int max_mem_len, int c, int t, int tc,
                                   const int32_t* pos0s, int pos_stride, float theta_base, loma_dtype dtype,
                                   float softmax_scale, unsigned flags, void* stream) {
    if (pos_stride < 0) return LOMA_ERR_INVALID_ARG;
    if (B > 0 && H > 0 && !pos0s) return LOMA_ERR_INVALID_ARG;
    if ((uintptr_t)pos0s & 3u) return LOMA_ERR_ALIGNMENT;
    RopeArgs rope;
    rope.on = 1; rope.pos_seq = pos0s; rope.stride = pos_stride;
    rope.log2_base = log2(theta_base > 0.f ? (double)theta_base : 10000.0);
    return loma_compress_step_ragged_impl(q_mem, k_mem, v_mem, k_cache, v_cache, o_mem, lse, B, H, D, cap, mem_lens,
                                          max_mem_len, c, t, tc, dtype, softmax_scale, flags, stream, rope);
}

int loma_selftest_bounded_wait(void* stream) {
    const int dc = check_device();
    if (dc != LOMA_OK) return dc;
    return launch_bounded_wait_selftest(static_cast<cudaStream_t>(stream)) == cudaSuccess ? LOMA_OK : LOMA_ERR_CUDA;
}

int loma_device_status(void* stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return LOMA_ERR_CUDA;
    int* w = device_status_word();
    if (!w) return LOMA_ERR_CUDA;
    int val = 0;
    if (cudaMemcpy(&val, w, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return LOMA_ERR_CUDA;
    if (val != 0) {
        const int zero = 0;
        if (cudaMemcpy(w, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return LOMA_ERR_CUDA;
    }
    return val;
}

}  // extern "C"
