// Backward of the zone-masked attention on the 5th-generation tensor cores (sm_100a):
// gradients of Eq. 7 along the paths of Section 4.4, with the tile plan of the forward.
//
// With P_ij = exp(scale q_i.k_j - lse_i) on the entries Eq. 2 allows, delta_i = dO_i.O_i and
// dA_ij = P_ij (dO_i.v_j - delta_i):   dQ = scale dA K,   dK = scale dA^T Q,   dV = P^T dO.
//
// dQ kernel.  One persistent CTA per SM works through query tiles (128 rows of a zone view, dealt
// longest first).  Q and dO of the tile stay in shared memory; K and V tiles of the keys the tile
// may see stream through a two-stage ring (TMA).  Per visited 64-key half ("event", see the
// forward kernel): S = Q K_h^T and dP = dO V_h^T (operands in shared memory, accumulators in two
// double-buffered 64-column TMEM regions each); the warpgroup (thread = query row = TMEM lane)
// turns them into dA, rounds it to bf16 and writes it back over S; dQ += dA K_h with dA read from
// TMEM and K_h as an MN-major shared operand.  Nothing is carried from event to event (lse and
// delta are inputs), so there is no rescaling.  Epilogue: scale, round to bf16, TMA store.
//
// dK/dV kernel.  The same machinery turned round: a CTA owns a key tile (K and V stay in shared
// memory, dK and dV accumulate in TMEM) and walks the query tiles that visit it (the plan read by
// key tile); Q and dO stream through the ring.  Per visited half of 64 query rows: S^T = K Q_h^T and
// dP^T = V dO_h^T; the warpgroup (thread = key row) writes P^T over S^T and dA^T over dP^T in bf16
// (lse and delta of the 128 query rows of the step are staged in shared memory); then
// dV += P^T dO_h and dK += dA^T Q_h with Q_h, dO_h as MN-major operands.
//
// Roles: warps 0-7 two warpgroups (each takes half of the columns of every event, and half of the
// epilogue), warp 8 TMA producer (one lane), warps 9 and 10 MMA issuers (warp-uniform control flow, one
// elected lane issues; warp 9 the score products, warp 10 the accumulating products).  Every mbarrier wait is bounded; on expiry the CTA
// records LOMA_ERR_TIMEOUT, every role leaves its loop, TMEM is freed and the kernel returns.
#include "tcgen05_common.cuh"

namespace loma {
// Work item -> key tile rank and (batch, head) in the dK/dV kernel, whose tiles are dealt statically.  Pair by
// pair, as in the other kernels, while a pair has fewer key tiles than there are CTAs (several pairs are then in
// flight and each pair's Q / dO stay in L2: 3 % on the 4608-token layout); one rank for every pair before the
// next rank otherwise: with 544 key tiles per pair of which 32 are a hundred times longer than the rest, the
// static deal is only even when those come first for all pairs (2 % on the 69632-token layout).
__device__ __forceinline__ void split_key_work(const FwdParams& p, int w, int& rank, int& bh) {
    if (p.total_tiles <= (int)gridDim.x) { split_work(p, w, rank, bh); return; }
    rank = fdiv(w, p.dBH);
    bh = w - rank * p.BH;
}
}  // namespace loma


namespace loma {

struct BwdMaps {
    CUtensorMap q[4], k[4], v[4], g[4], dq[4];   // g = dO
};

struct BwdParams {
    FwdParams f;
    const float* lse_in;   // [B*H, S] natural-log normaliser of the forward
    const float* delta;    // [B*H, S] dO_i . O_i
    float scale;
};

constexpr int BWD_THREADS = 352;   // two warpgroups, one TMA warp, two MMA warps
constexpr int BWD_NBAR = 13;

template <int D>
struct BwdDqSmem {
    static constexpr int PANELS = D / 64;
    static constexpr int PANEL_BYTES = 128 * 128;
    static constexpr int TILE_BYTES = PANELS * PANEL_BYTES;
    static constexpr int Q_OFF = 0;
    static constexpr int G_OFF = TILE_BYTES;
    static constexpr int KV_OFF = 2 * TILE_BYTES;          // stage s: K at KV_OFF + 2*s*TILE, V one tile further
    static constexpr int O_OFF = 6 * TILE_BYTES;           // two 64-column staging panels of the output, one per warpgroup
    static constexpr int TOTAL = 6 * TILE_BYTES + 2 * PANEL_BYTES;
};

// ------------------------------------------------------------------ delta_i = dO_i . O_i
template <int D>
__global__ void __launch_bounds__(256)
bwd_delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ g, float* __restrict__ delta, int H,
                 int S, int64_t sb, int64_t sh, int64_t ss) {
    // D/8 lanes per row, 16 bytes per lane
    constexpr int LPR = D / 8, RPW = 32 / LPR;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = (blockIdx.x * 8 + warp) * RPW + lane / LPR;
    const int bh = blockIdx.y, b = bh / H, h = bh - b * H;
    float acc = 0.f;
    if (row < S) {
        const int64_t off = (int64_t)b * sb + (int64_t)h * sh + (int64_t)row * ss + (lane % LPR) * 8;
        const uint4 a = __ldg(reinterpret_cast<const uint4*>(o + off)), c = __ldg(reinterpret_cast<const uint4*>(g + off));
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) acc = fmaf(bf16lo(aw[e]), bf16lo(cw[e]), fmaf(bf16hi(aw[e]), bf16hi(cw[e]), acc));
    }
#pragma unroll
    for (int m = LPR / 2; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
    if (row < S && lane % LPR == 0) delta[(int64_t)bh * S + row] = acc;
}

// ------------------------------------------------------------------ dQ
template <int D>
__global__ void __launch_bounds__(BWD_THREADS, 1)
masked_attn_bwd_dq_tc_kernel(const __grid_constant__ BwdMaps maps, const BwdParams bp) {
    using SM = BwdDqSmem<D>;
    constexpr int PANELS = SM::PANELS;
    const FwdParams& p = bp.f;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[BWD_NBAR];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    enum { B_QF = 0, B_QE = 1, B_KVF = 2, B_KVE = 4, B_SF = 6, B_PF = 8, B_DQ = 10, B_DA = 11 };
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < BWD_NBAR; ++i) mbar_init(bar(i), (i == B_PF || i == B_PF + 1) ? 256 : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // zero the operand buffers once: rows a TMA box does not cover keep finite contents
    for (int i = threadIdx.x; i < SM::TOTAL / 16; i += BWD_THREADS) reinterpret_cast<uint4*>(smem_gen)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // TMEM columns: S buffers at 0 and 64, dP buffers at 128 and 192, dQ accumulator at 256
    const uint32_t tmem = tmem_slot;
    volatile int* abortp = &abort_flag;

    const int total_work = p.total_tiles * p.BH;
    const int nstreams = gridDim.x;
    const int sid = blockIdx.x;
    auto tile_of_round = [&](int r) { return r * nstreams + ((r & 1) ? nstreams - 1 - sid : sid); };
    auto kv_off = [&](int stage) { return (uint32_t)(SM::KV_OFF + stage * 2 * SM::TILE_BYTES); };

    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t gs = 0, tcount = 0;
            bool ok = true;
            for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r), ++tcount) {
                int rank, bh;
                split_work(p, w, rank, bh);
                const int bi = fdiv(bh, p.dH), hi = bh - bi * p.H;
                TileDesc td;
                decode_tile(p, rank, td);
                const View& qv = p.view[td.view];
                if (tcount > 0) ok = mbar_wait(bar(B_QE), (tcount - 1) & 1, abortp, p.status);
                if (!ok) break;
                mbar_expect_tx(bar(B_QF), 2 * qv.R * qv.CH * 128 * PANELS);
                for (int pn = 0; pn < PANELS; ++pn) {
                    tma_load_5d(smem_base + SM::Q_OFF + pn * SM::PANEL_BYTES, &maps.q[td.view], bar(B_QF), pn * 64, td.r0, td.c0,
                                hi, bi);
                    tma_load_5d(smem_base + SM::G_OFF + pn * SM::PANEL_BYTES, &maps.g[td.view], bar(B_QF), pn * 64, td.r0, td.c0,
                                hi, bi);
                }
                for (int j = 0; j < td.nsteps; ++j, ++gs) {
                    KTile kt;
                    step_ktile(p, td, j, kt);
                    const View& kv = p.view[kt.view];
                    const int stage = gs & 1;
                    ok = mbar_wait(bar(B_KVE + stage), ((gs >> 1) & 1) ^ 1, abortp, p.status);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_KVF + stage), 2 * kv.R * kv.CH * 128 * PANELS);
                    for (int pn = 0; pn < PANELS; ++pn) {
                        tma_load_5d(smem_base + kv_off(stage) + pn * SM::PANEL_BYTES, &maps.k[kt.view], bar(B_KVF + stage), pn * 64,
                                    kt.r0, kt.c0, hi, bi);
                        tma_load_5d(smem_base + kv_off(stage) + SM::TILE_BYTES + pn * SM::PANEL_BYTES, &maps.v[kt.view],
                                    bar(B_KVF + stage), pn * 64, kt.r0, kt.c0, hi, bi);
                    }
                }
            }
            if (!ok) {
                // leaving early: give copies already in flight a bounded time to land in this CTA's shared memory
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000ll) {}
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ MMA issuer A: the score products
        // Two warps issue: this one S and dP, warp 10 the dQ accumulation.  An issuing thread runs in
        // step with the tensor pipe (the instruction queue is short), so whatever integer work one warp
        // does between its instructions is covered by the other warp's instructions in the pipe.
        constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
        uint32_t gs = 0, tcount = 0, ge = 0;
        bool ok = true;
        const uint64_t qd = smem_desc(smem_base + SM::Q_OFF, 16, 1024);
        const uint64_t gd = smem_desc(smem_base + SM::G_OFF, 16, 1024);
        for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r), ++tcount) {
            int rank, bh_;
            split_work(p, w, rank, bh_);
            TileDesc td;
            decode_tile(p, rank, td);
            const HalfMasks hm = tile_half_masks(p, td, lane);
            const int nsteps = td.nsteps;
            ok = __all_sync(0xffffffffu, mbar_wait(bar(B_QF), tcount & 1, abortp, p.status));
            HalfWalk sw;
            for (sw.start(hm); ok && !sw.done(nsteps); sw.next(hm), ++ge) {
                const uint32_t step = gs + sw.j;
                const int b = ge & 1, h = sw.h, stage = step & 1;
                if (sw.first_of_step(hm))
                    ok = __all_sync(0xffffffffu, mbar_wait(bar(B_KVF + stage), (step >> 1) & 1, abortp, p.status));
                // buffer b is free once the dQ product of event ge - 2 has read its dA out of it
                if (ok && ge >= 2) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_DA + b), ((ge - 2) >> 1) & 1, abortp, p.status));
                if (!ok) break;
                tc_fence_after();
                const bool last_of_tile = sw.last_of_step(hm) && sw.j == nsteps - 1;
                // S = Q K_h^T and dP = dO V_h^T of keys [64h, 64h+64) of the staged tiles -> buffers b
                if (elect_one()) {
                    const uint64_t kd = smem_desc(smem_base + kv_off(stage), 16, 1024);
                    const uint64_t vd = smem_desc(smem_base + kv_off(stage) + SM::TILE_BYTES, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint64_t off = (uint64_t)(((kk >> 2) * SM::PANEL_BYTES + (kk & 3) * 32) >> 4);
                        mma_ss(tmem + b * 64, qd + off, kd + off + (uint64_t)((h * 8192) >> 4), IDESC_S, kk > 0);
                    }
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint64_t off = (uint64_t)(((kk >> 2) * SM::PANEL_BYTES + (kk & 3) * 32) >> 4);
                        mma_ss(tmem + 128 + b * 64, gd + off, vd + off + (uint64_t)((h * 8192) >> 4), IDESC_S, kk > 0);
                    }
                    tc_commit(bar(B_SF + b));
                    if (last_of_tile) tc_commit(bar(B_QE));   // Q and dO are not read again in this tile
                }
                __syncwarp();
            }
            gs += td.nsteps;
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------ MMA issuer B: the dQ accumulation
        constexpr uint32_t IDESC_DQ =
            (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)D >> 3) << 17) | ((128u >> 4) << 24);
        uint32_t gs = 0, ge = 0;
        bool ok = true;
        for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r)) {
            int rank, bh_;
            split_work(p, w, rank, bh_);
            TileDesc td;
            decode_tile(p, rank, td);
            const HalfMasks hm = tile_half_masks(p, td, lane);
            const int nsteps = td.nsteps;
            bool first = true;
            HalfWalk pw;
            for (pw.start(hm); ok && !pw.done(nsteps); pw.next(hm), ++ge, first = false) {
                const int b = ge & 1, h = pw.h, stage = (gs + pw.j) & 1;
                const bool los = pw.last_of_step(hm), lot = los && pw.j == nsteps - 1;
                ok = __all_sync(0xffffffffu, mbar_wait(bar(B_PF + b), (ge >> 1) & 1, abortp, p.status));
                if (!ok) break;
                tc_fence_after();
                // dQ += dA K[64h .. 64h+63]: dA (bf16) read from TMEM over the S buffer (16 keys = 8 columns; keys
                // 0-31 at columns 0-15, keys 32-63 at columns 32-47: each warpgroup writes inside the columns it
                // read), K as an MN-major operand
                if (elect_one()) {
                    const uint64_t kmn = smem_desc(smem_base + kv_off(stage), SM::PANEL_BYTES, 1024);
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        mma_ts(tmem + 256, tmem + b * 64 + (k4 >> 1) * 32 + (k4 & 1) * 8, kmn + (uint64_t)(((h * 4 + k4) * 2048) >> 4),
                               IDESC_DQ, !first || (k4 > 0));
                    tc_commit(bar(B_DA + b));
                    if (los) tc_commit(bar(B_KVE + stage));
                    if (lot) tc_commit(bar(B_DQ));
                }
                __syncwarp();
            }
            gs += td.nsteps;
        }
    } else {
        // ------------------------------------------------------------ two warpgroups: dA, epilogue
        // thread = query row = TMEM lane; warpgroup wg takes columns [32 wg, 32 wg + 32) of every event
        const int rr = threadIdx.x & 127, wg = warp >> 2;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t ge = 0, tcount = 0;
        bool ok = true;
        bool store_pending = false;
        for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r), ++tcount) {
            int rank, bh;
            split_work(p, w, rank, bh);
            const int bi = fdiv(bh, p.dH), hi = bh - bi * p.H;
            TileDesc td;
            decode_tile(p, rank, td);
            const View& qv = p.view[td.view];
            const int rsub = fdiv(rr, qv.dR);
            const int ro = td.r0 + (rr - rsub * qv.R);
            const int rc = td.a0 + rsub;
            const bool row_valid = (rr < qv.R * qv.CH) && (rc <= td.a1) && (ro < qv.Z);
            float neg_lse2 = 0.f, dl = 0.f;
            if (row_valid) {
                const int64_t idx = (int64_t)bh * p.S + (int64_t)rc * p.s + qv.zone_row0 + ro;
                neg_lse2 = -bp.lse_in[idx] * 1.4426950408889634f;
                dl = bp.delta[idx];
            }
            const HalfMasks hm = tile_half_masks(p, td, lane);
            HalfWalk hw;
            int lo = 0, hi2 = 0;
            for (hw.start(hm); ok && !hw.done(td.nsteps); hw.next(hm), ++ge) {
                if (hw.first_of_step(hm)) {
                    KTile kt;
                    step_ktile(p, td, hw.j, kt);
                    row_interval(p.view[kt.view], kt, rc, ro, rr, row_valid, lo, hi2, p.view[kt.view].diag);
                }
                const int b = ge & 1;
                const int lo_h = lo - 64 * hw.h;
                const uint32_t span = (uint32_t)(hi2 - lo);
                ok = __all_sync(0xffffffffu, mbar_wait(bar(B_SF + b), (ge >> 1) & 1, abortp, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t s_addr = lane_addr + b * 64, g_addr = lane_addr + 128 + b * 64;
                // no row of this warp sees any of its 32 columns of this half: dA = 0, nothing to read
                if (__all_sync(0xffffffffu, hi2 - 64 * hw.h <= wg * 32 || lo_h >= wg * 32 + 32 || hi2 <= lo)) {
                    uint32_t z[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) z[e] = 0u;
                    tmem_st16(s_addr + wg * 32, z);
                } else {
                    const int c = wg;
                    uint32_t s[32], g[32], pk[16];
                    tmem_ld32(s_addr + c * 32, s);
                    tmem_ld32(g_addr + c * 32, g);
                    tmem_wait_ld();
                    // every row of this warp sees all 32 columns: no compare per entry
                    const bool full = __all_sync(0xffffffffu, lo_h <= c * 32 && hi2 - 64 * hw.h >= c * 32 + 32);
                    const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nl2 = pack2(neg_lse2, neg_lse2), ndl2 = pack2(-dl, -dl);
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float x0, x1, d0, d1;
                        unpack2(fma2(pack2(__uint_as_float(s[e]), __uint_as_float(s[e + 1])), sc2, nl2), x0, x1);
                        unpack2(add2(pack2(__uint_as_float(g[e]), __uint_as_float(g[e + 1])), ndl2), d0, d1);
                        float p0 = fast_ex2(x0), p1 = fast_ex2(x1);
                        if (!full) {
                            if ((uint32_t)(c * 32 + e - lo_h) >= span) p0 = 0.f;
                            if ((uint32_t)(c * 32 + e + 1 - lo_h) >= span) p1 = 0.f;
                        }
                        pk[e >> 1] = pack_bf16(p0 * d0, p1 * d1);
                    }
                    tmem_st16(s_addr + c * 32, pk);   // dA over the scores this warpgroup has just read: 32 keys -> 16 columns
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar(B_PF + b));
            }
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_DQ), tcount & 1, abortp, p.status));
            if (ok) tc_fence_after();

            // epilogue: scale, round to bf16, stage in shared memory, TMA store.  Warpgroup wg takes
            // the output columns [64 wg, 64 wg + 64) (its own staging panel, its own named barrier).
            // Every thread of a warpgroup reaches the first barrier for every tile it started; it
            // also makes giving up a uniform decision.
            uint8_t* orow = smem_gen + SM::O_OFF + wg * SM::PANEL_BYTES + rr * 128;
            bool give_up = false;
            if (wg < PANELS) {
                const int pn = wg;
                if (rr == 0 && store_pending) tma_store_wait_read();   // the staging panel is free again
                uint32_t any_bad;
                asm volatile(
                    "{\n.reg .pred p, q;\nsetp.ne.u32 p, %1, 0;\nbar.red.or.pred q, %2, 128, p;\nselp.u32 %0, 1, 0, q;\n}"
                    : "=r"(any_bad)
                    : "r"((uint32_t)(ok ? 0 : 1)), "r"(1 + wg)
                    : "memory");
                if (any_bad) give_up = true;
                if (!give_up) {
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t x[32];
                        tmem_ld32(lane_addr + 256 + pn * 64 + c * 32, x);
                        tmem_wait_ld();
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const int ci = c * 4 + q4;       // 16-byte chunk of the 128-byte panel row
                            uint4 u;
                            u.x = pack_bf16(__uint_as_float(x[q4 * 8 + 0]) * bp.scale, __uint_as_float(x[q4 * 8 + 1]) * bp.scale);
                            u.y = pack_bf16(__uint_as_float(x[q4 * 8 + 2]) * bp.scale, __uint_as_float(x[q4 * 8 + 3]) * bp.scale);
                            u.z = pack_bf16(__uint_as_float(x[q4 * 8 + 4]) * bp.scale, __uint_as_float(x[q4 * 8 + 5]) * bp.scale);
                            u.w = pack_bf16(__uint_as_float(x[q4 * 8 + 6]) * bp.scale, __uint_as_float(x[q4 * 8 + 7]) * bp.scale);
                            *reinterpret_cast<uint4*>(orow + ((ci ^ (rr & 7)) << 4)) = u;
                        }
                    }
                    fence_async_smem();
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + wg) : "memory");
                    if (rr == 0) {
                        tma_store_5d(&maps.dq[td.view], smem_base + SM::O_OFF + wg * SM::PANEL_BYTES, pn * 64, td.r0, td.c0, hi, bi);
                        tma_store_commit();
                        store_pending = true;
                    }
                }
            } else if (!ok) {
                give_up = true;
            }
            if (give_up) { ok = false; break; }
            tc_fence_before();
        }
        if (rr == 0 && store_pending) tma_store_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    }
}

// ------------------------------------------------------------------ dK, dV
struct BwdKvMaps {
    CUtensorMap q[4], k[4], v[4], g[4], dk[4], dv[4];
};

__device__ __forceinline__ HalfMasks key_tile_half_masks(const FwdParams& p, const KeyTileDesc& kd, int lane) {
    HalfMasks hm;
    hm.m[0] = hm.m[1] = 0;
    for (int base = 0; base < kd.nsteps && base < 64; base += 32) {
        const int j = base + lane;
        const unsigned v = j < kd.nsteps ? visited_qhalves(p, kd, j) : 0u;
        hm.m[0] |= (unsigned long long)__ballot_sync(0xffffffffu, v & 1u) << base;
        hm.m[1] |= (unsigned long long)__ballot_sync(0xffffffffu, v & 2u) << base;
    }
    return hm;
}

template <int D>
__global__ void __launch_bounds__(BWD_THREADS, 1)
masked_attn_bwd_dkv_tc_kernel(const __grid_constant__ BwdKvMaps maps, const BwdParams bp) {
    using SM = BwdDqSmem<D>;   // same footprint: two resident tiles, a two-stage ring of tile pairs, one staging panel
    constexpr int PANELS = SM::PANELS;
    constexpr int K_OFF = SM::Q_OFF, V_OFF = SM::G_OFF;
    const FwdParams& p = bp.f;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[BWD_NBAR];
    __shared__ __align__(16) float lse2_s[128];   // -lse * log2(e) and delta of the 128 query rows of the current step
    __shared__ __align__(16) float dl_s[128];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    enum { B_KVF = 0, B_DONE = 1, B_QGF = 2, B_QGE = 4, B_SF = 6, B_PF = 8, B_DA = 10 };
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < BWD_NBAR; ++i) mbar_init(bar(i), (i == B_PF || i == B_PF + 1) ? 256 : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = threadIdx.x; i < SM::TOTAL / 16; i += BWD_THREADS) reinterpret_cast<uint4*>(smem_gen)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // TMEM columns: S^T buffers at 0 and 64, dP^T buffers at 128 and 192, dK accumulator at 256, dV at 384
    const uint32_t tmem = tmem_slot;
    volatile int* abortp = &abort_flag;

    const int total_work = p.total_tiles * p.BH;
    const int nstreams = gridDim.x;
    const int sid = blockIdx.x;
    auto tile_of_round = [&](int r) { return r * nstreams + ((r & 1) ? nstreams - 1 - sid : sid); };
    auto ring_off = [&](int stage) { return (uint32_t)(SM::KV_OFF + stage * 2 * SM::TILE_BYTES); };   // Q, then dO

    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t gs = 0, tcount = 0;
            bool ok = true;
            for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r), ++tcount) {
                int rank, bh;
                split_key_work(p, w, rank, bh);
                const int bi = fdiv(bh, p.dH), hi = bh - bi * p.H;
                KeyTileDesc kd;
                decode_key_tile(p, rank, kd);
                const View& kv = p.view[kd.view];
                if (tcount > 0) ok = mbar_wait(bar(B_DONE), (tcount - 1) & 1, abortp, p.status);
                if (!ok) break;
                mbar_expect_tx(bar(B_KVF), 2 * kv.R * kv.CH * 128 * PANELS);
                for (int pn = 0; pn < PANELS; ++pn) {
                    tma_load_5d(smem_base + K_OFF + pn * SM::PANEL_BYTES, &maps.k[kd.view], bar(B_KVF), pn * 64, kd.r0, kd.c0, hi, bi);
                    tma_load_5d(smem_base + V_OFF + pn * SM::PANEL_BYTES, &maps.v[kd.view], bar(B_KVF), pn * 64, kd.r0, kd.c0, hi, bi);
                }
                for (int j = 0; j < kd.nsteps; ++j, ++gs) {
                    QTile qt;
                    step_qtile(p, kd, j, qt);
                    const View& qv = p.view[qt.view];
                    const int stage = gs & 1;
                    ok = mbar_wait(bar(B_QGE + stage), ((gs >> 1) & 1) ^ 1, abortp, p.status);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_QGF + stage), 2 * qv.R * qv.CH * 128 * PANELS);
                    for (int pn = 0; pn < PANELS; ++pn) {
                        tma_load_5d(smem_base + ring_off(stage) + pn * SM::PANEL_BYTES, &maps.q[qt.view], bar(B_QGF + stage), pn * 64,
                                    qt.r0, qt.c0, hi, bi);
                        tma_load_5d(smem_base + ring_off(stage) + SM::TILE_BYTES + pn * SM::PANEL_BYTES, &maps.g[qt.view],
                                    bar(B_QGF + stage), pn * 64, qt.r0, qt.c0, hi, bi);
                    }
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000ll) {}
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ MMA issuer A: the score products
        // (two issuing warps, as in the dQ kernel: this one S^T and dP^T, warp 10 the dV and dK accumulation)
        constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
        uint32_t gs = 0, tcount = 0, ge = 0;
        bool ok = true;
        const uint64_t kd_ = smem_desc(smem_base + K_OFF, 16, 1024);
        const uint64_t vd_ = smem_desc(smem_base + V_OFF, 16, 1024);
        for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r), ++tcount) {
            int rank, bh_;
            split_key_work(p, w, rank, bh_);
            KeyTileDesc kd;
            decode_key_tile(p, rank, kd);
            const HalfMasks hm = key_tile_half_masks(p, kd, lane);
            const int nsteps = kd.nsteps;
            ok = __all_sync(0xffffffffu, mbar_wait(bar(B_KVF), tcount & 1, abortp, p.status));
            HalfWalk sw;
            for (sw.start(hm); ok && !sw.done(nsteps); sw.next(hm), ++ge) {
                const uint32_t step = gs + sw.j;
                const int b = ge & 1, h = sw.h, stage = step & 1;
                if (sw.first_of_step(hm))
                    ok = __all_sync(0xffffffffu, mbar_wait(bar(B_QGF + stage), (step >> 1) & 1, abortp, p.status));
                // buffers b are free once the accumulation of event ge - 2 has read P^T and dA^T out of them
                if (ok && ge >= 2) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_DA + b), ((ge - 2) >> 1) & 1, abortp, p.status));
                if (!ok) break;
                tc_fence_after();
                // S^T = K Q_h^T and dP^T = V dO_h^T for query rows [64h, 64h+64) of the staged tiles -> buffers b
                if (elect_one()) {
                    const uint64_t qd = smem_desc(smem_base + ring_off(stage), 16, 1024);
                    const uint64_t gd = smem_desc(smem_base + ring_off(stage) + SM::TILE_BYTES, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint64_t off = (uint64_t)(((kk >> 2) * SM::PANEL_BYTES + (kk & 3) * 32) >> 4);
                        mma_ss(tmem + b * 64, kd_ + off, qd + off + (uint64_t)((h * 8192) >> 4), IDESC_S, kk > 0);
                    }
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint64_t off = (uint64_t)(((kk >> 2) * SM::PANEL_BYTES + (kk & 3) * 32) >> 4);
                        mma_ss(tmem + 128 + b * 64, vd_ + off, gd + off + (uint64_t)((h * 8192) >> 4), IDESC_S, kk > 0);
                    }
                    tc_commit(bar(B_SF + b));
                }
                __syncwarp();
            }
            gs += kd.nsteps;
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------ MMA issuer B: the dV and dK accumulation
        constexpr uint32_t IDESC_ACC =
            (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)D >> 3) << 17) | ((128u >> 4) << 24);
        uint32_t gs = 0, ge = 0;
        bool ok = true;
        for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r)) {
            int rank, bh_;
            split_key_work(p, w, rank, bh_);
            KeyTileDesc kd;
            decode_key_tile(p, rank, kd);
            const HalfMasks hm = key_tile_half_masks(p, kd, lane);
            const int nsteps = kd.nsteps;
            bool first = true;
            HalfWalk pw;
            for (pw.start(hm); ok && !pw.done(nsteps); pw.next(hm), ++ge, first = false) {
                const int b = ge & 1, h = pw.h, stage = (gs + pw.j) & 1;
                const bool los = pw.last_of_step(hm), lot = los && pw.j == nsteps - 1;
                ok = __all_sync(0xffffffffu, mbar_wait(bar(B_PF + b), (ge >> 1) & 1, abortp, p.status));
                if (!ok) break;
                tc_fence_after();
                // dV += P^T dO_h and dK += dA^T Q_h: P^T and dA^T (bf16) read from TMEM, dO_h and Q_h as MN-major operands
                if (elect_one()) {
                    const uint64_t qmn = smem_desc(smem_base + ring_off(stage), SM::PANEL_BYTES, 1024);
                    const uint64_t gmn = smem_desc(smem_base + ring_off(stage) + SM::TILE_BYTES, SM::PANEL_BYTES, 1024);
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        mma_ts(tmem + 384, tmem + b * 64 + (k4 >> 1) * 32 + (k4 & 1) * 8, gmn + (uint64_t)(((h * 4 + k4) * 2048) >> 4),
                               IDESC_ACC, !first || (k4 > 0));
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        mma_ts(tmem + 256, tmem + 128 + b * 64 + (k4 >> 1) * 32 + (k4 & 1) * 8,
                               qmn + (uint64_t)(((h * 4 + k4) * 2048) >> 4), IDESC_ACC, !first || (k4 > 0));
                    tc_commit(bar(B_DA + b));
                    if (los) tc_commit(bar(B_QGE + stage));
                    if (lot) tc_commit(bar(B_DONE));
                }
                __syncwarp();
            }
            gs += kd.nsteps;
        }
    } else {
        // ------------------------------------------------------------ two warpgroups: P^T, dA^T, epilogue
        // thread = key row = TMEM lane; warpgroup wg takes query rows [32 wg, 32 wg + 32) of every event
        const int kr = threadIdx.x & 127, wg = warp >> 2;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t ge = 0, gs = 0, tcount = 0;
        bool ok = true;
        bool store_pending = false;
        for (int r = 0, w = sid; w < total_work && ok; w = tile_of_round(++r), ++tcount) {
            int rank, bh;
            split_key_work(p, w, rank, bh);
            const int bi = fdiv(bh, p.dH), hi = bh - bi * p.H;
            KeyTileDesc kd;
            decode_key_tile(p, rank, kd);
            const View& kv = p.view[kd.view];
            const int ksub = fdiv(kr, kv.dR);
            const int ko = kd.r0 + (kr - ksub * kv.R);
            const int kc = kd.a0 + ksub;
            const bool key_valid = (kr < kv.R * kv.CH) && (kc <= kd.a1) && (ko < kv.Z);
            const HalfMasks hm = key_tile_half_masks(p, kd, lane);
            HalfWalk hw;
            int lo = 0, hi2 = 0;
            for (hw.start(hm); ok && !hw.done(kd.nsteps); hw.next(hm), ++ge) {
                if (hw.first_of_step(hm)) {
                    QTile qt;
                    step_qtile(p, kd, hw.j, qt);
                    const View& qv = p.view[qt.view];
                    col_interval(qv, qt, kc, ko, kr, key_valid, lo, hi2);
                    // this thread fetches lse and delta of query row `kr` of the step's tile for everybody
                    const int rsub = fdiv(kr, qv.dR);
                    const int ro = qt.r0 + (kr - rsub * qv.R);
                    const int rc = qt.a0 + rsub;
                    float nl = 0.f, dl = 0.f;
                    if ((kr < qv.R * qv.CH) && (rc <= qt.a1) && (ro < qv.Z)) {
                        const int64_t idx = (int64_t)bh * p.S + (int64_t)rc * p.s + qv.zone_row0 + ro;
                        nl = -bp.lse_in[idx] * 1.4426950408889634f;
                        dl = bp.delta[idx];
                    }
                    asm volatile("bar.sync 3, 256;" ::: "memory");   // everybody has finished with the previous step's values
                    if (wg == 0) {
                        lse2_s[kr] = nl;
                        dl_s[kr] = dl;
                    }
                    asm volatile("bar.sync 3, 256;" ::: "memory");
                }
                const int b = ge & 1;
                const int lo_h = lo - 64 * hw.h;
                const uint32_t span = (uint32_t)(hi2 - lo);
                ok = __all_sync(0xffffffffu, mbar_wait(bar(B_SF + b), (ge >> 1) & 1, abortp, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t s_addr = lane_addr + b * 64, g_addr = lane_addr + 128 + b * 64;
                // no key row of this warp is seen by any of its 32 query rows of this half: P^T = dA^T = 0
                if (__all_sync(0xffffffffu, hi2 - 64 * hw.h <= wg * 32 || lo_h >= wg * 32 + 32 || hi2 <= lo)) {
                    uint32_t z[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) z[e] = 0u;
                    tmem_st16(s_addr + wg * 32, z);
                    tmem_st16(g_addr + wg * 32, z);
                } else {
                    const int c = wg;
                    uint32_t s[32], g[32], ppk[16], dpk[16];
                    tmem_ld32(s_addr + c * 32, s);
                    tmem_ld32(g_addr + c * 32, g);
                    tmem_wait_ld();
                    const float4* nl4 = reinterpret_cast<const float4*>(&lse2_s[64 * hw.h + c * 32]);
                    const float4* dl4 = reinterpret_cast<const float4*>(&dl_s[64 * hw.h + c * 32]);
                    const bool full = __all_sync(0xffffffffu, lo_h <= c * 32 && hi2 - 64 * hw.h >= c * 32 + 32);
                    const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2);
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        const float4 nl = nl4[e >> 2], dl = dl4[e >> 2];
                        float x[4], d[4];
                        unpack2(fma2(pack2(__uint_as_float(s[e]), __uint_as_float(s[e + 1])), sc2, pack2(nl.x, nl.y)), x[0], x[1]);
                        unpack2(fma2(pack2(__uint_as_float(s[e + 2]), __uint_as_float(s[e + 3])), sc2, pack2(nl.z, nl.w)), x[2], x[3]);
                        d[0] = __uint_as_float(g[e]) - dl.x; d[1] = __uint_as_float(g[e + 1]) - dl.y;
                        d[2] = __uint_as_float(g[e + 2]) - dl.z; d[3] = __uint_as_float(g[e + 3]) - dl.w;
                        float pr[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            pr[u] = fast_ex2(x[u]);
                            if (!full && (uint32_t)(c * 32 + e + u - lo_h) >= span) pr[u] = 0.f;
                        }
                        ppk[e >> 1] = pack_bf16(pr[0], pr[1]);
                        ppk[(e >> 1) + 1] = pack_bf16(pr[2], pr[3]);
                        dpk[e >> 1] = pack_bf16(pr[0] * d[0], pr[1] * d[1]);
                        dpk[(e >> 1) + 1] = pack_bf16(pr[2] * d[2], pr[3] * d[3]);
                    }
                    tmem_st16(s_addr + c * 32, ppk);   // P^T over the scores this warpgroup has just read: 32 query rows -> 16 columns
                    tmem_st16(g_addr + c * 32, dpk);   // dA^T over dP^T, likewise
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar(B_PF + b));
            }
            gs += kd.nsteps;
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_DONE), tcount & 1, abortp, p.status));
            if (ok) tc_fence_after();

            // epilogue: warpgroup 0 stores dK (scaled), warpgroup 1 stores dV, each rounded to bf16 and
            // taken 64 columns at a time through its own staging panel and named barrier
            uint8_t* orow = smem_gen + SM::O_OFF + wg * SM::PANEL_BYTES + kr * 128;
            const float mul = wg == 0 ? bp.scale : 1.f;
            bool give_up = false;
#pragma unroll
            for (int pn = 0; pn < PANELS; ++pn) {
                if (kr == 0 && store_pending) tma_store_wait_read();
                if (pn == 0) {
                    uint32_t any_bad;
                    asm volatile(
                        "{\n.reg .pred p, q;\nsetp.ne.u32 p, %1, 0;\nbar.red.or.pred q, %2, 128, p;\nselp.u32 %0, 1, 0, q;\n}"
                        : "=r"(any_bad)
                        : "r"((uint32_t)(ok ? 0 : 1)), "r"(1 + wg)
                        : "memory");
                    if (any_bad) { give_up = true; break; }
                } else {
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + wg) : "memory");
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t x[32];
                    tmem_ld32(lane_addr + 256 + wg * 128 + pn * 64 + c * 32, x);
                    tmem_wait_ld();
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const int ci = c * 4 + q4;
                        uint4 u;
                        u.x = pack_bf16(__uint_as_float(x[q4 * 8 + 0]) * mul, __uint_as_float(x[q4 * 8 + 1]) * mul);
                        u.y = pack_bf16(__uint_as_float(x[q4 * 8 + 2]) * mul, __uint_as_float(x[q4 * 8 + 3]) * mul);
                        u.z = pack_bf16(__uint_as_float(x[q4 * 8 + 4]) * mul, __uint_as_float(x[q4 * 8 + 5]) * mul);
                        u.w = pack_bf16(__uint_as_float(x[q4 * 8 + 6]) * mul, __uint_as_float(x[q4 * 8 + 7]) * mul);
                        *reinterpret_cast<uint4*>(orow + ((ci ^ (kr & 7)) << 4)) = u;
                    }
                }
                fence_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(1 + wg) : "memory");
                if (kr == 0) {
                    tma_store_5d(wg == 0 ? &maps.dk[kd.view] : &maps.dv[kd.view], smem_base + SM::O_OFF + wg * SM::PANEL_BYTES, pn * 64,
                                 kd.r0, kd.c0, hi, bi);
                    tma_store_commit();
                    store_pending = true;
                }
            }
            if (give_up) { ok = false; break; }
            tc_fence_before();
        }
        if (kr == 0 && store_pending) tma_store_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    }
}

// ------------------------------------------------------------------ host side
struct BwdMapCacheKey {
    const void *q, *k, *v, *g, *dq;
    int B, H, D, n, c, t, tail;
    unsigned flags;
    int64_t sb, sh, ss;
    bool operator==(const BwdMapCacheKey& r) const {
        return q == r.q && k == r.k && v == r.v && g == r.g && dq == r.dq && B == r.B && H == r.H && D == r.D && n == r.n &&
               c == r.c && t == r.t && tail == r.tail && flags == r.flags && sb == r.sb && sh == r.sh && ss == r.ss;
    }
};

// delta (all rows) and dQ on the tensor cores.  Returns cudaErrorNotSupported when this path cannot
// take the call (the caller then uses the CUDA-core kernels).
cudaError_t launch_masked_attn_bwd_dq_tc(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                         const float* lse, void* dq, float* delta, int B, int H, int D, const Layout& L,
                                         int64_t sb, int64_t sh, int64_t ss, float scale, cudaStream_t st) {
    if (!encode_fn()) return cudaErrorNotSupported;
    if (L.t > 256 * 128 || L.tc > (1 << 24)) return cudaErrorNotSupported;

    BwdParams bp{};
    make_plan(L, B, H, &bp.f);
    bp.f.scale_log2 = scale * 1.4426950408889634f;
    bp.f.status = device_status_word();
    if (!bp.f.status) return cudaErrorUnknown;
    if ((int64_t)bp.f.total_tiles * bp.f.BH > 0x7fffffffll) return cudaErrorNotSupported;
    bp.lse_in = lse;
    bp.delta = delta;
    bp.scale = scale;

    static std::mutex mu;
    static BwdMapCacheKey cached_key{};
    static BwdMaps cached_maps;
    static bool have_cache = false;
    BwdMaps maps;
    {
        std::lock_guard<std::mutex> lock(mu);
        BwdMapCacheKey key{q, k, v, d_o, dq, B, H, D, L.n_chunks, L.c, L.t, L.tail_read, L.flags, sb, sh, ss};
        if (!(have_cache && key == cached_key)) {
            BwdMaps mnew{};
            const void* bases[5] = {q, k, v, d_o, dq};
            CUtensorMap* arrs[5] = {mnew.q, mnew.k, mnew.v, mnew.g, mnew.dq};
            for (int ti = 0; ti < 5; ++ti) {
                for (int vi = 0; vi < 4; ++vi) {
                    const View& vw = bp.f.view[vi];
                    if (vw.ntiles == 0) continue;
                    const int64_t row0 = (vi == V_TAIL) ? (int64_t)L.n_chunks * L.s : vw.zone_row0;
                    if (!encode_view(&arrs[ti][vi], bases[ti], vw, D, B, H, row0, sb, sh, ss, L.s)) return cudaErrorNotSupported;
                }
            }
            cached_maps = mnew;
            cached_key = key;
            have_cache = true;
        }
        maps = cached_maps;
    }

    static int sm_count[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (sm_count[dev] == 0) {
        int sms = 0;
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(masked_attn_bwd_dq_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 BwdDqSmem<128>::TOTAL + 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(masked_attn_bwd_dq_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 BwdDqSmem<64>::TOTAL + 1024);
        if (e != cudaSuccess) return e;
        sm_count[dev] = sms;
    }
    const int sms = sm_count[dev];

    // delta: 8 warps per CTA, 32 / (D/8) rows per warp
    const int rows_per_cta = 8 * (32 / (D / 8));
    dim3 dgrid((L.S + rows_per_cta - 1) / rows_per_cta, B * H);
    if (D == 128)
        bwd_delta_kernel<128><<<dgrid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o),
                                                     delta, H, L.S, sb, sh, ss);
    else
        bwd_delta_kernel<64><<<dgrid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o),
                                                    delta, H, L.S, sb, sh, ss);

    const int64_t work = (int64_t)bp.f.total_tiles * bp.f.BH;
    const int grid = (int)(work < sms ? work : sms);
    if (D == 128)
        masked_attn_bwd_dq_tc_kernel<128><<<grid, BWD_THREADS, BwdDqSmem<128>::TOTAL + 1024, st>>>(maps, bp);
    else
        masked_attn_bwd_dq_tc_kernel<64><<<grid, BWD_THREADS, BwdDqSmem<64>::TOTAL + 1024, st>>>(maps, bp);
    count_launches(2);
    return cudaGetLastError();
}

struct BwdKvMapCacheKey {
    const void *q, *k, *v, *g, *dk, *dv;
    int B, H, D, n, c, t, tail;
    unsigned flags;
    int64_t sb, sh, ss;
    bool operator==(const BwdKvMapCacheKey& r) const {
        return q == r.q && k == r.k && v == r.v && g == r.g && dk == r.dk && dv == r.dv && B == r.B && H == r.H && D == r.D &&
               n == r.n && c == r.c && t == r.t && tail == r.tail && flags == r.flags && sb == r.sb && sh == r.sh && ss == r.ss;
    }
};

// dK and dV on the tensor cores; delta must already be in place (launch_masked_attn_bwd_dq_tc writes it).
cudaError_t launch_masked_attn_bwd_dkv_tc(const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                                          const float* delta, void* dk, void* dv, int B, int H, int D, const Layout& L,
                                          int64_t sb, int64_t sh, int64_t ss, float scale, cudaStream_t st) {
    if (!encode_fn()) return cudaErrorNotSupported;
    if (L.t > 256 * 128 || L.tc > (1 << 24)) return cudaErrorNotSupported;
    BwdParams bp{};
    make_plan(L, B, H, &bp.f);
    bp.f.scale_log2 = scale * 1.4426950408889634f;
    bp.f.status = device_status_word();
    if (!bp.f.status) return cudaErrorUnknown;
    if ((int64_t)bp.f.total_tiles * bp.f.BH > 0x7fffffffll) return cudaErrorNotSupported;
    bp.lse_in = lse;
    bp.delta = delta;
    bp.scale = scale;

    static std::mutex mu;
    static BwdKvMapCacheKey cached_key{};
    static BwdKvMaps cached_maps;
    static bool have_cache = false;
    BwdKvMaps maps;
    {
        std::lock_guard<std::mutex> lock(mu);
        BwdKvMapCacheKey key{q, k, v, d_o, dk, dv, B, H, D, L.n_chunks, L.c, L.t, L.tail_read, L.flags, sb, sh, ss};
        if (!(have_cache && key == cached_key)) {
            BwdKvMaps mnew{};
            const void* bases[6] = {q, k, v, d_o, dk, dv};
            CUtensorMap* arrs[6] = {mnew.q, mnew.k, mnew.v, mnew.g, mnew.dk, mnew.dv};
            for (int ti = 0; ti < 6; ++ti) {
                for (int vi = 0; vi < 4; ++vi) {
                    const View& vw = bp.f.view[vi];
                    if (vw.ntiles == 0) continue;
                    const int64_t row0 = (vi == V_TAIL) ? (int64_t)L.n_chunks * L.s : vw.zone_row0;
                    if (!encode_view(&arrs[ti][vi], bases[ti], vw, D, B, H, row0, sb, sh, ss, L.s)) return cudaErrorNotSupported;
                }
            }
            cached_maps = mnew;
            cached_key = key;
            have_cache = true;
        }
        maps = cached_maps;
    }

    static int sm_count[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (sm_count[dev] == 0) {
        int sms = 0;
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(masked_attn_bwd_dkv_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 BwdDqSmem<128>::TOTAL + 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(masked_attn_bwd_dkv_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 BwdDqSmem<64>::TOTAL + 1024);
        if (e != cudaSuccess) return e;
        sm_count[dev] = sms;
    }
    const int sms = sm_count[dev];
    static_assert(BwdDqSmem<128>::TOTAL + 1024 + 1536 <= 227 * 1024, "dynamic + static shared memory of the backward kernels");
    const int64_t work = (int64_t)bp.f.total_tiles * bp.f.BH;
    const int grid = (int)(work < sms ? work : sms);
    if (D == 128)
        masked_attn_bwd_dkv_tc_kernel<128><<<grid, BWD_THREADS, BwdDqSmem<128>::TOTAL + 1024, st>>>(maps, bp);
    else
        masked_attn_bwd_dkv_tc_kernel<64><<<grid, BWD_THREADS, BwdDqSmem<64>::TOTAL + 1024, st>>>(maps, bp);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace loma
