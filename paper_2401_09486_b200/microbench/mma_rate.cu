// Microbenchmark: clocks per tcgen05.mma (kind::f16, M = 128, K = 16) for N = 64, 128, 256, with both operands in shared
// memory (SS) or A in TMEM (TS).  One CTA, one issuing warp, 64 x 8 back-to-back instructions on zeroed operands; the
// issue time (until the last instruction is accepted) and the completion time (until the commit arrives) are reported
// per instruction.  Build and run on a B200:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I include -I paper_2401_09486_b200/csrc \
//        -o mma_rate paper_2401_09486_b200/microbench/mma_rate.cu && ./mma_rate
#include <cstdio>
#include "tcgen05_common.cuh"
using namespace loma;
template <int N, bool TS>
__global__ void __launch_bounds__(128, 1) rate_kernel(long long* out, int reps) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_s;
    __shared__ uint32_t tmem_slot;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (smem_base - smem_u32(smem_raw));
    for (int i = threadIdx.x; i < (32768 + 65536) / 16; i += 128) reinterpret_cast<uint4*>(gen)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar_s), 1); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
    const int warp = threadIdx.x >> 5;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before(); __syncthreads(); tc_fence_after();
    const uint32_t tmem = tmem_slot;
    if (warp == 1) {
        constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)N >> 3) << 17) | ((128u >> 4) << 24);
        const uint64_t ad = smem_desc(smem_base, 16, 1024);
        const uint64_t bd = smem_desc(smem_base + 32768, 16, 1024);
        long long t0 = 0, t1 = 0, t2 = 0;
        uint32_t ph = 0;
        for (int round = 0; round < 3; ++round) {
            t0 = clock64();
            if (elect_one()) {
                for (int r = 0; r < reps; ++r) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint64_t off = (uint64_t)(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
                        if (TS) mma_ts(tmem, tmem + 256 + kk * 8, bd + off, IDESC, 1);
                        else mma_ss(tmem, ad + off, bd + off, IDESC, 1);
                    }
                }
                tc_commit(smem_u32(&bar_s));
            }
            __syncwarp();
            t1 = clock64();
            while (!mbar_try_wait(smem_u32(&bar_s), ph)) { if (clock64() - t1 > 2000000000ll) break; }
            ph ^= 1;
            t2 = clock64();
        }
        if ((threadIdx.x & 31) == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
    }
    tc_fence_before(); __syncthreads();
    if (warp == 0) { tc_fence_after(); asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"(512) : "memory"); }
}
template <int N, bool TS> void run(const char* name) {
    long long* d; cudaMalloc(&d, 16); long long h[2];
    const int reps = 64; const int smem = 32768 + 65536 + 1024;
    cudaFuncSetAttribute(rate_kernel<N, TS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    rate_kernel<N, TS><<<1, 128, smem>>>(d, reps);
    cudaError_t e = cudaDeviceSynchronize();
    cudaMemcpy(h, d, 16, cudaMemcpyDeviceToHost);
    printf("%s N=%d: %s issue %.1f clk/mma, complete %.1f clk/mma (ideal %.0f)\n", name, N, cudaGetErrorString(e), h[0] / (reps * 8.0), h[1] / (reps * 8.0), 128.0 * N * 16 * 2 / 8192);
    cudaFree(d);
}
int main() {
    run<64, false>("SS"); run<128, false>("SS"); run<256, false>("SS");
    run<64, true>("TS"); run<128, true>("TS"); run<256, true>("TS");
    return 0;
}
