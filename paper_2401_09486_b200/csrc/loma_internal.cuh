// Internal declarations shared by the translation units of libloma.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "loma.h"

namespace loma {

// ---- layout parameters handed to kernels ---------------------------------
struct Layout {
    int n_chunks;   // complete chunks
    int c, t, tc;   // tc = c*t
    int s;          // chunk length 2*tc + t (0 when t == 0)
    int tail_read;  // trailing reading rows
    int S;          // n_chunks*s + tail_read
    unsigned flags;
};

// ---- one row of the laid-out sequence (shared by the index-map and rotary kernels) ----
struct RowInfo {
    int chunk, zone, offset, src, pos;
};

// Row i of the laid-out sequence -> its chunk, zone, offset, source token and
// position id.  Rows beyond the last complete chunk are reading rows of chunk
// n_chunks.  Memory position ids follow Eq. 14 with the chunk start at y*tc.
__host__ __device__ inline RowInfo layout_row(int i, int n_chunks, int c, int t, int s) {
    const int tc = c * t;   // s: chunk length, 2*tc + t, or tc + t in the layout without repetition zones
    RowInfo r;
    if (s == 0 || i >= n_chunks * s) {
        r.chunk = n_chunks;
        r.zone = LOMA_ZONE_READ;
        r.offset = i - n_chunks * s;
    } else {
        r.chunk = i / s;
        const int rem = i - r.chunk * s;
        if (rem < tc) {
            r.zone = LOMA_ZONE_READ;
            r.offset = rem;
        } else if (rem < tc + t) {
            r.zone = LOMA_ZONE_MEM;
            r.offset = rem - tc;
        } else {
            r.zone = LOMA_ZONE_REP;
            r.offset = rem - tc - t;
        }
    }
    if (r.zone == LOMA_ZONE_MEM) {
        r.src = -1;
        r.pos = r.chunk * tc + (r.offset + 1) * c - 1;
    } else {
        r.src = r.chunk * tc + r.offset;
        r.pos = r.src;
    }
    return r;
}

// ---- paged cache: a pool of pages [n_pages, H, page_size, D]; table[b * max_pages + p] = page of sequence b's p-th block.
// table == NULL means a contiguous cache [B, H, cap, D].
struct Paging {
    const int32_t* table = nullptr;
    int max_pages = 0, log2_ps = 0, n_pages = 0;
};

// ---- rotary embedding fused into the generation steps (Section 4.5; Appendix A position ids) -------------
// pos0 + j * stride is the position id of row j of the call (decode: one row; compress: the t memory rows,
// Eq. 14 with pos0 = y*tc + c - 1, stride = c, or the contiguous ids with pos0 = mem_len, stride = 1).
struct RopeArgs {
    int on = 0;
    int pos0 = 0, stride = 0;
    const int32_t* pos_seq = nullptr;   // [device] one pos0 per sequence of the batch (ragged batches), or NULL: pos0 for all
    double log2_base = 0.0;   // log2 of the base (10000 by default)
};

#ifdef __CUDACC__
// cos and sin of the rotation angle of feature pair (d, d + D/2) at position pos: pos * base^(-2d/D).  The angle
// is formed and reduced to [-pi, pi] in double (ids reach tens of thousands, where a float angle has lost the
// digits the fp32 bar needs); cos/sin of the reduced angle in float are good to ~2e-7.
__device__ __forceinline__ void rope_cos_sin(int pos, int d, int D, double log2_base, float& c, float& s) {
    const double theta = exp2(-log2_base * (2.0 * d / D));
    double a = (double)pos * theta;
    a -= 6.283185307179586476925 * rint(a * 0.15915494309189533577);
    sincosf((float)a, &s, &c);
}
#endif

// ---- launchers (each defined in its own .cu) ------------------------------
cudaError_t launch_layout_index(const Layout& L, int32_t* chunk, int32_t* zone, int32_t* offset,
                                int32_t* src, int32_t* pos, cudaStream_t st);
cudaError_t launch_generation_index(int n_tokens, int c, int t, int32_t* slot, int32_t* pos,
                                    int32_t* comp, cudaStream_t st);
cudaError_t launch_prefill_cache(const void* k, const void* v, void* kc, void* vc, int B, int H, int row_bytes, int cap,
                                 const Layout& L, int64_t sb_bytes, int64_t sh_bytes, int64_t ss_bytes, cudaStream_t st);
void host_layout_index(const Layout& L, int32_t* chunk, int32_t* zone, int32_t* offset, int32_t* src,
                       int32_t* pos);
void host_generation_index(int n_tokens, int c, int t, int32_t* slot, int32_t* pos, int32_t* comp);

cudaError_t launch_masked_attn_generic(const void* q, const void* k, const void* v, void* o, float* lse,
                                       int B, int H, int D, const Layout& L,
                                       int64_t sb, int64_t sh, int64_t ss,
                                       loma_dtype dt, float scale, cudaStream_t st);

// gradients of the masked forward on CUDA cores; delta: B*H*S floats of scratch (row sums dO.O).
// parts: bit 0 = delta and dQ, bit 1 = dK and dV (needs delta)
cudaError_t launch_masked_attn_bwd_generic(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                           const float* lse, void* dq, void* dk, void* dv, float* delta, int B, int H,
                                           int D, const Layout& L, int64_t sb, int64_t sh, int64_t ss, loma_dtype dt,
                                           float scale, int parts, cudaStream_t st);
// bf16 on tcgen05 (attn_bwd_tcgen05.cu): delta for every row, and dQ; cudaErrorNotSupported = use the generic kernels
cudaError_t launch_masked_attn_bwd_dq_tc(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                         const float* lse, void* dq, float* delta, int B, int H, int D, const Layout& L,
                                         int64_t sb, int64_t sh, int64_t ss, float scale, cudaStream_t st);
cudaError_t launch_masked_attn_bwd_dkv_tc(const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                                          const float* delta, void* dk, void* dv, int B, int H, int D, const Layout& L,
                                          int64_t sb, int64_t sh, int64_t ss, float scale, cudaStream_t st);

// tcgen05 / TMEM / TMA masked forward (attn_tcgen05.cu); cudaErrorNotSupported = use the generic kernel
cudaError_t launch_masked_attn_tc(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int D,
                                  const Layout& L, int64_t sb, int64_t sh, int64_t ss, float scale, cudaStream_t st);

// l new tokens over a cache that already holds their K/V at [cache_len, cache_len + l) (attn_tcgen05.cu)
cudaError_t launch_prefill_attn_tc(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse, int B,
                                   int H, int D, int l, int cap, int cache_len, const int32_t* cache_lens,
                                   const Paging& pg, float scale, cudaStream_t st);
// the same on CUDA cores (any l, fp32 or bf16), and the bit-exact append that precedes both (attn_generic.cu)
cudaError_t launch_prefill_attn_generic(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                                        int B, int H, int D, int l, int cap, int cache_len, const int32_t* lens,
                                        const Paging& pg, loma_dtype dt, float scale, cudaStream_t st);
cudaError_t launch_cache_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache, int B, int H,
                                int row_bytes, int l, int cap, int cache_len, const int32_t* lens, const Paging& pg,
                                int pad_to, bool copy_k, cudaStream_t st);
cudaError_t launch_prefill_rope(const void* q, const void* k_new, void* q_rot, void* k_cache, int B, int H, int D, int l,
                                int cap, int cache_len, const int32_t* lens, const Paging& pg, const RopeArgs& rope,
                                loma_dtype dt, cudaStream_t st);

void plan_coverage_host(const Layout& L, uint8_t* counts);          // tile_plan_host.cu
void prefill_plan_coverage_host(int l, int cache_len, uint8_t* counts);
void plan_coverage_by_key_host(const Layout& L, uint8_t* counts);   // the plan read by key tile (backward)

cudaError_t launch_bounded_wait_selftest(cudaStream_t st);   // attn_tcgen05.cu

cudaError_t launch_decode_generic(const void* q, const void* k_new, const void* v_new,
                                  void* k_cache, void* v_cache, void* o, float* lse,
                                  int B, int H, int D, int cap, int cache_len, const int32_t* lens,
                                  loma_dtype dt, float scale, const Paging& pg, cudaStream_t st,
                                  const RopeArgs& rope = RopeArgs{});

// bf16 split-KV decode (decode_splitkv.cu)
size_t decode_workspace_bytes(int BH, int D, int total_keys);
cudaError_t launch_decode_bf16(const void* q, const void* k_new, const void* v_new, void* k_cache,
                               void* v_cache, void* o, float* lse, int B, int H, int D, int cap, int cache_len,
                               const int32_t* lens, float scale, void* ws, const Paging& pg,
                               cudaStream_t st, const RopeArgs& rope = RopeArgs{});   // lens: per-sequence lengths or NULL

size_t decode_static_scratch_bytes();
cudaError_t launch_decode_bf16_static(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                      void* v_cache, void* o, float* lse, int B, int H, int D, int cap,
                                      int cache_len, float scale, cudaStream_t st);

// bf16 compress step on warp-level tensor cores (compress_mma.cu); t <= 16
size_t compress_workspace_bytes(int BH, int D, int t, int mem_len, unsigned flags);
cudaError_t launch_compress_bf16(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache, void* v_cache,
                                 void* o_mem, float* lse, int B, int H, int D, int cap, int mem_len,
                                 const int32_t* mem_lens, int c, int t, unsigned flags, float scale, void* ws,
                                 const Paging& pg, cudaStream_t st,
                                 const RopeArgs& rope = RopeArgs{});   // mem_lens: per-sequence counts (default variant only) or NULL

cudaError_t launch_compress_generic(const void* q_mem, const void* k_mem, const void* v_mem,
                                    void* k_cache, void* v_cache, void* o_mem, float* lse,
                                    int B, int H, int D, int cap, int mem_len, const int32_t* mem_lens, int c, int t,
                                    loma_dtype dt, float scale, unsigned flags, const Paging& pg, cudaStream_t st,
                                    const RopeArgs& rope = RopeArgs{});

// rotary embedding of Q and K rows at the layout's position ids (rope.cu)
cudaError_t launch_rope(void* q, void* k, int B, int H, int D, const Layout& L, int64_t sb, int64_t sh, int64_t ss,
                        loma_dtype dt, double theta_base, int position_type, cudaStream_t st);

// ---- launch accounting -------------------------------------------------------
void count_launches(int n);   // called by every launcher with the number of kernels it enqueued

// ---- device status word (bounded waits report here) ------------------------
int* device_status_word();   // device address of the status word of the current device (NULL on failure)

// ---- small device helpers ---------------------------------------------------
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// two packed bf16 -> two floats (exact)
__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
    return *reinterpret_cast<uint32_t*>(&p);
}

}  // namespace loma
