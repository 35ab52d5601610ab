// Integer index maps of the LoMA layout (Section 4.1, Eq. 14) and of the
// generation-time cache (Section 3.1, Appendix A).  Pure integer work; the host
// and device versions use the same inline row functions.
#include "loma_internal.cuh"

namespace loma {

struct GenInfo {
    int slot, pos, comp;
};

// Generated token g -> cache slot it is appended at, its position id, and
// whether the tail is full (tc entries) once it has been appended.
__host__ __device__ inline GenInfo generation_row(int g, int c, int t) {
    GenInfo r;
    r.pos = g;
    if (t == 0) {
        r.slot = g;
        r.comp = 0;
    } else {
        const int tc = c * t;
        const int y = g / tc;
        const int o = g - y * tc;
        r.slot = y * t + o;
        r.comp = (o == tc - 1) ? 1 : 0;
    }
    return r;
}

__global__ void layout_index_kernel(int S, int n_chunks, int c, int t, int s, int32_t* chunk, int32_t* zone,
                                    int32_t* offset, int32_t* src, int32_t* pos) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= S) return;
    const RowInfo r = layout_row(i, n_chunks, c, t, s);
    if (chunk) chunk[i] = r.chunk;
    if (zone) zone[i] = r.zone;
    if (offset) offset[i] = r.offset;
    if (src) src[i] = r.src;
    if (pos) pos[i] = r.pos;
}

__global__ void generation_index_kernel(int n, int c, int t, int32_t* slot, int32_t* pos, int32_t* comp) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n) return;
    const GenInfo r = generation_row(g, c, t);
    if (slot) slot[g] = r.slot;
    if (pos) pos[g] = r.pos;
    if (comp) comp[g] = r.comp;
}

// Gather of the rows that survive in the cache (memory zones in order, then the reading tail):
// one CTA row of 16-byte vectors per (destination row, b*h); bit-exact copies.
__global__ void prefill_cache_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v, uint4* __restrict__ kc,
                                     uint4* __restrict__ vc, int H, int vec_per_row, int cap, int n_chunks, int t,
                                     int tc, int s, int n_rows, int64_t sb_v, int64_t sh_v, int64_t ss_v) {
    const int dst = blockIdx.x;                        // cache slot
    const int bh = blockIdx.y;
    const int b = bh / H, h = bh - b * H;
    // slot -> row of the laid-out sequence
    const int n_mem = n_chunks * t;
    const int64_t src = dst < n_mem ? (int64_t)(dst / t) * s + tc + (dst % t) : (int64_t)n_chunks * s + (dst - n_mem);
    const int64_t in = (int64_t)b * sb_v + (int64_t)h * sh_v + src * ss_v;
    const int64_t out = ((int64_t)bh * cap + dst) * vec_per_row;
    for (int e = threadIdx.x; e < vec_per_row; e += blockDim.x) {
        kc[out + e] = __ldg(k + in + e);
        vc[out + e] = __ldg(v + in + e);
    }
    (void)n_rows;
}

cudaError_t launch_prefill_cache(const void* k, const void* v, void* kc, void* vc, int B, int H, int row_bytes, int cap,
                                 const Layout& L, int64_t sb_bytes, int64_t sh_bytes, int64_t ss_bytes, cudaStream_t st) {
    const int n_rows = L.n_chunks * L.t + L.tail_read;
    if (n_rows == 0 || B * H == 0) return cudaSuccess;
    const int vec = row_bytes / 16;
    dim3 grid(n_rows, B * H);
    prefill_cache_kernel<<<grid, 32, 0, st>>>(static_cast<const uint4*>(k), static_cast<const uint4*>(v),
                                             static_cast<uint4*>(kc), static_cast<uint4*>(vc), H, vec, cap, L.n_chunks,
                                             L.t, L.tc, L.s, n_rows, sb_bytes / 16, sh_bytes / 16, ss_bytes / 16);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_layout_index(const Layout& L, int32_t* chunk, int32_t* zone, int32_t* offset,
                                int32_t* src, int32_t* pos, cudaStream_t st) {
    if (L.S == 0) return cudaSuccess;
    const int threads = 256;
    layout_index_kernel<<<(L.S + threads - 1) / threads, threads, 0, st>>>(L.S, L.n_chunks, L.c, L.t, L.s, chunk,
                                                                         zone, offset, src, pos);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_generation_index(int n_tokens, int c, int t, int32_t* slot, int32_t* pos,
                                    int32_t* comp, cudaStream_t st) {
    if (n_tokens == 0) return cudaSuccess;
    const int threads = 256;
    generation_index_kernel<<<(n_tokens + threads - 1) / threads, threads, 0, st>>>(n_tokens, c, t, slot, pos,
                                                                                  comp);
    count_launches(1);
    return cudaGetLastError();
}

void host_layout_index(const Layout& L, int32_t* chunk, int32_t* zone, int32_t* offset, int32_t* src,
                       int32_t* pos) {
    for (int i = 0; i < L.S; ++i) {
        const RowInfo r = layout_row(i, L.n_chunks, L.c, L.t, L.s);
        if (chunk) chunk[i] = r.chunk;
        if (zone) zone[i] = r.zone;
        if (offset) offset[i] = r.offset;
        if (src) src[i] = r.src;
        if (pos) pos[i] = r.pos;
    }
}

void host_generation_index(int n_tokens, int c, int t, int32_t* slot, int32_t* pos, int32_t* comp) {
    for (int g = 0; g < n_tokens; ++g) {
        const GenInfo r = generation_row(g, c, t);
        if (slot) slot[g] = r.slot;
        if (pos) pos[g] = r.pos;
        if (comp) comp[g] = r.comp;
    }
}

}  // namespace loma
