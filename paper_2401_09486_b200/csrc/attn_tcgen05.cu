// Zone-masked attention forward on the 5th-generation tensor cores (sm_100a):
// tcgen05.mma with TMEM accumulators, operands staged by TMA.
//
// The mask of Eq. 1-3 is never stored and never evaluated entry by entry.  The
// sequence is seen through four "zone views" -- reading, memory and repetition
// zones of the complete chunks, and the reading tail -- each a 5-D tensor
// (d, row in zone, chunk, head, batch) over the caller's Q/K/V/O.  A tile is
// 128 rows of one view: 128 consecutive rows of a zone when the zone is at
// least that long, otherwise the whole zone of as many consecutive chunks as
// fit (one TMA box gathers them into a dense tile).  For a query tile only the
// key tiles that hold an allowed entry are visited (everything else is
// skipped), and inside a visited tile the allowed columns of a row always form
// one interval [lo, hi), so the mask costs two compares per score at most:
//
//   reading rows    x memory tiles of earlier chunks   key chunk <  row chunk  (Eq. 3)
//   reading rows    x own reading zone                 causal                   (L of Eq. 1)
//   memory rows     x own reading and memory zone      key chunk == row chunk   (Eq. 1, row 2)
//   memory rows     x earlier memory zones             key chunk <= row chunk   (prior-memory flag)
//   repetition rows x own memory zone                  key chunk == row chunk   (Eq. 1, row 3)
//   repetition rows x themselves                       diagonal                 (I of Eq. 1)
//
// One CTA (384 threads) per SM, persistent.  A CTA runs two independent "streams": each stream
// owns a query tile at a time and has its own shared-memory buffers (Q, one K tile, one V tile,
// a 64-column output staging panel), its own quarter of TMEM (two 64-column score buffers and a
// 128-column output accumulator) and its own warps:
//   warps 0-3 / 4-7   softmax warpgroup of stream 0 / 1: thread = query row = TMEM lane.  The 128
//                     keys of a step are taken as two halves of 64: read the scores of a half,
//                     row maximum (three-input max), probabilities 2^(s*scale - ref) with packed
//                     two-wide fp32 FMA/ADD, bf16 P written back over the scores.  The output
//                     accumulates in TMEM; the reference maximum only moves, and the accumulator
//                     is only rescaled, when a row maximum has grown by more than 2^8.  Epilogue:
//                     normalise, round to bf16, stage 64 columns at a time, TMA store.
//   warp 8 / 9        TMA producer of stream 0 / 1 (one lane): Q per tile, K and V per step
//   warp 10 / 11      MMA issuer of stream 0 / 1: the warp's control flow is uniform and one
//                     elected lane issues, so descriptors stay in uniform registers (issuing from
//                     a divergent single-lane branch halved the tensor throughput).  Per step:
//                     S_h = Q K_h^T for both halves (operands in shared memory, N = 64), and
//                     O += P_h V_h with P read from TMEM and V as an MN-major shared operand.
//                     S_h of the next step is issued right after P_h V_h of this one, so the
//                     tensor pipe works on one half while the warpgroup works on the other.
// The two streams fill each other's waits (tensor latency, TMEM loads, epilogues).  Tiles are handed
// out at run time from one counter over a statically ordered list ((batch, head) by (batch, head), each
// pair's tiles longest first): a stream that finishes a tile draws the next (without a counter, see the host side, the tiles are
// dealt round robin).  Every mbarrier wait is bounded: on expiry the CTA records LOMA_ERR_TIMEOUT, all
// roles leave their loops, TMEM is freed and the kernel returns.
#include "tcgen05_common.cuh"

namespace loma {

struct TmaMaps {
    CUtensorMap q[4], k[4], v[4], o[4];
};

// ------------------------------------------------------------------ the kernel
constexpr int TC_THREADS = 384;   // 2 softmax warpgroups + 1 warpgroup with 2 TMA warps and 2 MMA warps
constexpr int TMEM_COLS = 512;
constexpr int NBAR = 14;          // mbarriers per stream

// Shared memory of one stream: Q tile, one K tile, one V tile, and a 64-column output staging panel.
template <int D>
struct TcSmem {
    static constexpr int PANELS = D / 64;
    static constexpr int PANEL_BYTES = 128 * 128;           // 128 rows x 64 bf16
    static constexpr int TILE_BYTES = PANELS * PANEL_BYTES; // one 128 x D tile
    static constexpr int Q_OFF = 0;
    static constexpr int K_OFF = TILE_BYTES;
    static constexpr int V_OFF = 2 * TILE_BYTES;
    static constexpr int O_OFF = 3 * TILE_BYTES;
    static constexpr int STREAM_BYTES = 3 * TILE_BYTES + PANEL_BYTES;
    static constexpr int TOTAL = 2 * STREAM_BYTES;
};

// RAGGED: the prefill plan of a batch whose sequences have their own cache lengths (p.prefill_lens); a kernel of
// its own so that the other plans carry none of it.
template <int D, bool RAGGED>
__global__ void __launch_bounds__(TC_THREADS, 1)
masked_attn_tc_kernel(const __grid_constant__ TmaMaps maps, const FwdParams p) {
    using SM = TcSmem<D>;
    constexpr int PANELS = SM::PANELS;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * NBAR];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int tile_ring_s[2][4];

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
    // which of the CTA's two independent streams this warp serves
    const int st = warp < 8 ? (warp >> 2) : (warp & 1);
    const uint32_t smem_base0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen0 = smem_raw + (smem_base0 - smem_u32(smem_raw));
    const uint32_t smem_base = smem_base0 + st * SM::STREAM_BYTES;
    uint8_t* smem_gen = smem_gen0 + st * SM::STREAM_BYTES;

    enum { B_QF = 0, B_QE = 1, B_KF = 2, B_KE = 3, B_VF = 4, B_VE = 5, B_SF = 6, B_PF = 8, B_OF = 10, B_TF = 12 };
    auto bar = [&](int i) { return smem_u32(&bars[st * NBAR + i]); };

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s2 = 0; s2 < 2; ++s2)
            for (int i = 0; i < NBAR; ++i) mbar_init(smem_u32(&bars[s2 * NBAR + i]), (i == B_PF || i == B_PF + 1) ? 128 : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // zero the operand buffers once: rows a TMA box does not cover keep finite contents
    for (int i = threadIdx.x; i < SM::TOTAL / 16; i += TC_THREADS)
        reinterpret_cast<uint4*>(smem_gen0)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    if (warp == 10) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot + st * 256;   // this stream's scores at +0, output accumulator at +128
    volatile int* abortp = &abort_flag;

    // Tiles are handed out from one counter, pair by pair and longest first inside a (batch, head): a stream
    // that finishes early simply takes the next one.  The stream's producer draws the number and posts it
    // in a four-slot ring (barrier B_TF + (n & 1), completion n >> 1, for the stream's n-th tile); the MMA
    // issuer and the warpgroup read it there.  A negative number ends the stream.  Which stream computes a
    // tile has no influence on the tile's result.
    const int total_work = p.total_tiles * p.BH;
    volatile int* tile_ring = tile_ring_s[st];
    auto next_tile = [&](uint32_t n, bool& ok_) -> int {   // called by whole warps
        ok_ = __all_sync(0xffffffffu, mbar_wait(bar(B_TF + (n & 1)), (n >> 1) & 1, abortp, p.status));
        return ok_ ? tile_ring[n & 3] : -1;
    };
    // ragged prompt pieces: batch element bi's own cache length (clamped to the length the plan was sized for)
    auto own_diag = [&](int bi) -> int {
        if (!RAGGED) return -1;
        return min(max(__ldg(p.prefill_lens + bi), 0), p.view[V_MEM].diag);
    };

    if (warp == 8 || warp == 9) {
        // ------------------------------------------------------------ TMA producer of stream st
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
        if (lane == 0) {
            uint32_t gs = 0, tcount = 0;
            bool ok = true;
            for (;; ++tcount) {
                // draw the stream's next tile and post it (a number past the end tells the other roles to stop)
                int w = p.sched ? (int)atomicAdd(p.sched, 1u) : (int)(2 * blockIdx.x + st + tcount * 2 * gridDim.x);
                if (w >= total_work || !ok) w = -1;
                tile_ring[tcount & 3] = w;
                __threadfence_block();
                mbar_arrive(bar(B_TF + (tcount & 1)));
                if (w < 0) break;
                int rank, bh;
                split_work(p, w, rank, bh);
                const int bi = fdiv(bh, p.dH), hi = bh - bi * p.H;
                TileDesc td;
                decode_tile(p, rank, td, own_diag(bi));
                const View& qv = p.view[td.view];
                if (tcount > 0) ok = mbar_wait(bar(B_QE), (tcount - 1) & 1, abortp, p.status);
                if (!ok) break;
                mbar_expect_tx(bar(B_QF), qv.R * qv.CH * 128 * PANELS);
                for (int pn = 0; pn < PANELS; ++pn)
                    tma_load_5d(smem_base + SM::Q_OFF + pn * SM::PANEL_BYTES, &maps.q[td.view], bar(B_QF), pn * 64, td.r0,
                                td.c0, hi, bi);
                for (int j = 0; j < td.nsteps; ++j, ++gs) {
                    KTile kt;
                    step_ktile(p, td, j, kt);
                    const View& kv = p.view[kt.view];
                    const uint32_t ph = gs & 1;
                    uint32_t bytes = kv.R * kv.CH * 128 * PANELS;
                    // where the key tile lies: (row, chunk, batch) of the caller's tensor, or, over a paged cache, (row in
                    // page, 0, page) of the pool -- pages hold a multiple of 128 rows, so a tile never straddles two
                    int kr = kt.r0, kc_ = kt.c0, kb = bi;
                    if (RAGGED && p.page_table) {
                        bytes = 128 * 128 * PANELS;   // the pool's box is always 128 rows, whatever the key view's length
                        kb = min(max(__ldg(p.page_table + (int64_t)bi * p.pt_stride + (kt.r0 >> p.log2_ps)), 0), p.n_pages - 1);
                        kr = kt.r0 & ((1 << p.log2_ps) - 1);
                        kc_ = 0;
                    }
                    ok = mbar_wait(bar(B_KE), ph ^ 1, abortp, p.status);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_KF), bytes);
                    for (int pn = 0; pn < PANELS; ++pn)
                        tma_load_5d(smem_base + SM::K_OFF + pn * SM::PANEL_BYTES, &maps.k[kt.view], bar(B_KF), pn * 64,
                                    kr, kc_, hi, kb);
                    ok = mbar_wait(bar(B_VE), ph ^ 1, abortp, p.status);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_VF), bytes);
                    for (int pn = 0; pn < PANELS; ++pn)
                        tma_load_5d(smem_base + SM::V_OFF + pn * SM::PANEL_BYTES, &maps.v[kt.view], bar(B_VF), pn * 64,
                                    kr, kc_, hi, kb);
                }
            }
            if (!ok) {
                // leaving early: give copies already in flight a bounded time to land in this CTA's shared memory
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000ll) {}
            }
        }
    } else if (warp >= 10) {
        // ------------------------------------------------------------ MMA issuer of stream st
        // All 32 lanes run the loops (warp-uniform); one elected lane issues the instructions.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;" ::: "memory");
        {
            // instruction descriptors: fp32 accumulate, bf16 x bf16, M = 128
            constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
            constexpr uint32_t IDESC_PV =
                (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)D >> 3) << 17) | ((128u >> 4) << 24);
            uint32_t gs = 0, tcount = 0;
            bool ok = true;
            const uint64_t qd = smem_desc(smem_base + SM::Q_OFF, 16, 1024);
            const uint64_t kd = smem_desc(smem_base + SM::K_OFF, 16, 1024);
            const uint64_t vd = smem_desc(smem_base + SM::V_OFF, SM::PANEL_BYTES, 1024);
            // Visited halves ("events") are numbered ge = 0, 1, 2, ... across all tiles of the stream.
            // Event ge uses score buffer ge & 1 and the barriers B_SF/B_PF/B_OF + (ge & 1), whose
            // completion number ge >> 1 gives the parity to wait for.  K/V buffers go by step (gs).
            // scores of keys [64h, 64h+64) of the staged key tile -> score buffer b (64 columns)
            auto issue_s = [&](int b, int h, bool last_of_step, bool last_of_tile) {
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        // descriptor start addresses are in 16-byte units; 64 key rows are 8192 bytes further
                        const uint64_t off = (uint64_t)(((kk >> 2) * SM::PANEL_BYTES + (kk & 3) * 32) >> 4);
                        mma_ss(tmem + b * 64, qd + off, kd + off + (uint64_t)((h * 8192) >> 4), IDESC_S, kk > 0);
                    }
                    tc_commit(bar(B_SF + b));
                    if (last_of_step) tc_commit(bar(B_KE));
                    if (last_of_tile) tc_commit(bar(B_QE));   // every score product of the tile has been issued
                }
                __syncwarp();
            };
            // O += P V[64h .. 64h+63]: four instructions of 16 keys, P read from TMEM over score buffer b
            auto issue_pv = [&](int b, int h, bool first, bool last_of_step) {
                if (elect_one()) {
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        mma_ts(tmem + 128, tmem + b * 64 + k4 * 8, vd + (uint64_t)(((h * 4 + k4) * 2048) >> 4), IDESC_PV,
                               !first || (k4 > 0));
                    tc_commit(bar(B_OF + b));   // one barrier per buffer: each completes once per event
                    if (last_of_step) tc_commit(bar(B_VE));
                }
                __syncwarp();
            };
            uint32_t ge_s = 0, ge_p = 0;   // events whose scores / whose P.V have been issued
            for (;; ++tcount) {
                const int w = next_tile(tcount, ok);
                if (w < 0) break;
                int rank, bh_m;
                split_work(p, w, rank, bh_m);
                TileDesc td;
                const int dg = own_diag(fdiv(bh_m, p.dH));
                decode_tile(p, rank, td, dg);
                const HalfMasks hm = tile_half_masks(p, td, lane, dg);
                const int nsteps = td.nsteps;
                HalfWalk sw, pw;
                sw.start(hm);
                pw.start(hm);
                ok = __all_sync(0xffffffffu, mbar_wait(bar(B_QF), tcount & 1, abortp, p.status));
                if (!ok) break;
                // the score products run two events ahead of the P.V products
                auto next_scores = [&]() {
                    if (sw.first_of_step(hm)) {
                        ok = __all_sync(0xffffffffu, mbar_wait(bar(B_KF), (gs + sw.j) & 1, abortp, p.status));
                        if (!ok) return;
                    }
                    tc_fence_after();
                    const bool los = sw.last_of_step(hm);
                    issue_s(ge_s & 1, sw.h, los, los && sw.j == nsteps - 1);
                    ++ge_s;
                    sw.next(hm);
                };
                next_scores();
                if (ok && !sw.done(nsteps)) next_scores();
                bool first = true;
                while (ok && !pw.done(nsteps)) {
                    const int b = ge_p & 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar(B_PF + b), (ge_p >> 1) & 1, abortp, p.status));
                    if (ok && pw.first_of_step(hm))
                        ok = __all_sync(0xffffffffu, mbar_wait(bar(B_VF), (gs + pw.j) & 1, abortp, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(b, pw.h, first, pw.last_of_step(hm));
                    first = false;
                    ++ge_p;
                    if (!sw.done(nsteps)) next_scores();
                    pw.next(hm);
                }
                gs += td.nsteps;
            }
        }
    } else {
        // ------------------------------------------------------------ softmax + epilogue of stream st (128 threads)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 232;" ::: "memory");
        const int rr = threadIdx.x & 127;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t s_addr = lane_addr, o_addr = lane_addr + 128;
        uint32_t ge = 0;   // visited halves so far (see the MMA issuer)
        bool ok = true;
        bool store_pending = false;
        // Everything this thread needs to know about a tile.  The next tile is decoded while the last
        // product of the current one drains, so the decode's chain of dependent loads and integer
        // arithmetic stays off the path between two tiles.
        struct TileCtx {
            TileDesc td;
            HalfMasks hm;
            int bh, bi, hi, ro, rc, zone_row0, diag;
            bool row_valid;
        };
        auto decode_ctx = [&](int w, TileCtx& c) {
            int rank;
            split_work(p, w, rank, c.bh);
            c.bi = fdiv(c.bh, p.dH);
            c.hi = c.bh - c.bi * p.H;
            c.diag = own_diag(c.bi);
            decode_tile(p, rank, c.td, c.diag);
            const View& qv = p.view[c.td.view];
            const int rsub = fdiv(rr, qv.dR);
            c.ro = c.td.r0 + (rr - rsub * qv.R);
            c.rc = c.td.a0 + rsub;
            c.zone_row0 = qv.zone_row0;
            c.row_valid = (rr < qv.R * qv.CH) && (c.rc <= c.td.a1) && (c.ro < qv.Z);
            c.hm = tile_half_masks(p, c.td, lane, c.diag);
        };
        TileCtx cur, nxt;
        uint32_t tcount = 0;
        int w_cur = next_tile(0, ok), w_next = -1;
        if (w_cur >= 0) decode_ctx(w_cur, cur);
        for (; w_cur >= 0 && ok; w_cur = w_next, cur = nxt, ++tcount) {
            const TileDesc& td = cur.td;
            const HalfMasks hm = cur.hm;
            const int bh = cur.bh, bi = cur.bi, hi = cur.hi, ro = cur.ro, rc = cur.rc;
            const bool row_valid = cur.row_valid;

            // Running reference maximum (exp2 domain) and row sum.  The reference only moves
            // when the row maximum has grown by more than 2^8 since it was set; then the
            // output accumulator in TMEM is rescaled once.  Probabilities stay below 2^8.
            float m_used = -INFINITY, l = 0.f;

            HalfWalk hw;
            bool first = true;
            int lo = 0, hi2 = 0;
            for (hw.start(hm); ok && !hw.done(td.nsteps); hw.next(hm), ++ge, first = false) {
                if (hw.first_of_step(hm)) {
                    KTile kt;
                    step_ktile(p, td, hw.j, kt);
                    row_interval(p.view[kt.view], kt, rc, ro, rr, row_valid, lo, hi2, RAGGED ? cur.diag : p.view[kt.view].diag);
                }
                // One visited half of a key tile (64 keys) per pass, in score buffer ge & 1: the tensor
                // pipe works on the other buffer while this warpgroup works on this one.
                {
                    const int b = ge & 1;
                    const int lo_h = lo - 64 * hw.h;                  // allowed columns of this half: [lo_h, lo_h + span)
                    const uint32_t span = (uint32_t)(hi2 - lo);
                    const int hi_h = hi2 - 64 * hw.h;
                    const bool full = __all_sync(0xffffffffu, lo_h <= 0 && hi_h >= 64);
                    // no row of this warp has an allowed column in this half (the other warps of the tile do):
                    // e.g. three of the four warps of a memory-zone tile at every reading half it visits
                    const bool none = __all_sync(0xffffffffu, hi_h <= 0 || lo_h >= 64 || hi2 <= lo);
                    ok = __all_sync(0xffffffffu, mbar_wait(bar(B_SF + b), (ge >> 1) & 1, abortp, p.status));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sh_addr = s_addr + b * 64;
                    if (none) {
                        // probabilities of zero for the warp's rows; the running maximum and sum stay as they are
                        uint32_t z[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) z[e] = 0u;
                        tmem_st16(sh_addr, z);
                        tmem_st16(sh_addr + 16, z);
                        tmem_wait_st();
                        tc_fence_before();
                        mbar_arrive(bar(B_PF + b));
                        continue;
                    }
                    uint32_t s[64];
                    tmem_ld32(sh_addr, s);
                    tmem_ld32(sh_addr + 32, s + 32);
                    tmem_wait_ld();
                    if (!full) {
                        if (__all_sync(0xffffffffu, lo_h <= 0)) {
                            // only an upper bound in this warp (causal and chunk-prefix masks): one compare per score
#pragma unroll
                            for (int e = 0; e < 64; ++e)
                                if (e >= hi_h) s[e] = 0xff800000u;   // -inf: blocked for this row
                        } else {
#pragma unroll
                            for (int e = 0; e < 64; ++e)
                                if ((uint32_t)(e - lo_h) >= span) s[e] = 0xff800000u;
                        }
                    }
                    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                    for (int e = 0; e < 64; e += 8) {
                        mx0 = max3(mx0, __uint_as_float(s[e]), __uint_as_float(s[e + 1]));
                        mx1 = max3(mx1, __uint_as_float(s[e + 2]), __uint_as_float(s[e + 3]));
                        mx2 = max3(mx2, __uint_as_float(s[e + 4]), __uint_as_float(s[e + 5]));
                        mx3 = max3(mx3, __uint_as_float(s[e + 6]), __uint_as_float(s[e + 7]));
                    }
                    const float mrow = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
                    const bool need = mrow > m_used + 8.f;
                    if (!first && __any_sync(0xffffffffu, need)) {
                        // rescale the accumulated output: wait until the previous event's P.V has landed in TMEM
                        ok = __all_sync(0xffffffffu,
                                        mbar_wait(bar(B_OF + ((ge - 1) & 1)), ((ge - 1) >> 1) & 1, abortp, p.status));
                        if (!ok) break;
                        tc_fence_after();
                        const float alpha = need ? fast_ex2(m_used - mrow) : 1.f;
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t r[32];
                            tmem_ld32(o_addr + c * 32, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                            tmem_st32(o_addr + c * 32, r);
                        }
                        l *= alpha;
                    }
                    if (need) m_used = mrow;
                    const float neg_ref = (m_used == -INFINITY) ? 0.f : -m_used;
                    const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nr2 = pack2(neg_ref, neg_ref);
                    uint64_t lsa = pack2(0.f, 0.f), lsb = lsa;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t pk[16];
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            float x0, x1, x2, x3;
                            unpack2(fma2(pack2(__uint_as_float(s[c * 32 + e]), __uint_as_float(s[c * 32 + e + 1])), sc2, nr2), x0, x1);
                            unpack2(fma2(pack2(__uint_as_float(s[c * 32 + e + 2]), __uint_as_float(s[c * 32 + e + 3])), sc2, nr2), x2, x3);
                            const float p0 = fast_ex2(x0), p1 = fast_ex2(x1), p2 = fast_ex2(x2), p3 = fast_ex2(x3);
                            lsa = add2(lsa, pack2(p0, p1));
                            lsb = add2(lsb, pack2(p2, p3));
                            pk[e >> 1] = pack_bf16(p0, p1);
                            pk[(e >> 1) + 1] = pack_bf16(p2, p3);
                        }
                        tmem_st16(sh_addr + c * 16, pk);   // P over the scores: 32 keys -> 16 columns
                    }
                    {
                        float a0, a1, b0, b1;
                        unpack2(lsa, a0, a1);
                        unpack2(lsb, b0, b1);
                        l += (a0 + a1) + (b0 + b1);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(bar(B_PF + b));
                }
            }
            {
                bool got = true;
                w_next = next_tile(tcount + 1, got);
                if (!got) ok = false;
                if (w_next >= 0) decode_ctx(w_next, nxt);
            }
            // the last P.V of the tile belongs to event ge - 1 (products complete in issue order)
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_OF + ((ge - 1) & 1)), ((ge - 1) >> 1) & 1, abortp, p.status));
            if (ok) tc_fence_after();

            // epilogue: normalise, round to bf16, stage 64 output columns at a time in shared
            // memory, TMA store.  A panel's 64 columns are fetched from TMEM with one wait and packed
            // before the thread that issued the previous panel's store waits for that store to have
            // read the staging panel, so the wait is covered by the fetch.  Every thread of the
            // warpgroup reaches the first barrier for every tile it started; it also makes giving up
            // a uniform decision.
            const float inv = 1.f / l;
            uint8_t* orow = smem_gen + SM::O_OFF + rr * 128;
            bool give_up = false;
#pragma unroll
            for (int pn = 0; pn < PANELS; ++pn) {
                uint32_t pk[32];
                {
                    uint32_t r[64];
                    tmem_ld32(o_addr + pn * 64, r);
                    tmem_ld32(o_addr + pn * 64 + 32, r + 32);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        pk[e] = pack_bf16(__uint_as_float(r[2 * e]) * inv, __uint_as_float(r[2 * e + 1]) * inv);
                }
                if (rr == 0 && store_pending) tma_store_wait_read();   // the staging panel is free again
                if (pn == 0) {
                    uint32_t any_bad;
                    asm volatile(
                        "{\n.reg .pred p, q;\nsetp.ne.u32 p, %1, 0;\nbar.red.or.pred q, %2, 128, p;\nselp.u32 %0, 1, 0, q;\n}"
                        : "=r"(any_bad)
                        : "r"((uint32_t)(ok ? 0 : 1)), "r"(1 + st)
                        : "memory");
                    if (any_bad) { give_up = true; break; }
                } else {
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + st) : "memory");
                }
#pragma unroll
                for (int ci = 0; ci < 8; ++ci)           // 16-byte chunk of the 128-byte panel row
                    *reinterpret_cast<uint4*>(orow + ((ci ^ (rr & 7)) << 4)) =
                        make_uint4(pk[ci * 4], pk[ci * 4 + 1], pk[ci * 4 + 2], pk[ci * 4 + 3]);
                fence_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(1 + st) : "memory");
                if (rr == 0) {
                    tma_store_5d(&maps.o[td.view], smem_base + SM::O_OFF, pn * 64, td.r0, td.c0, hi, bi);
                    tma_store_commit();
                    store_pending = true;
                }
            }
            if (give_up) { ok = false; break; }
            tc_fence_before();
            if (p.lse && row_valid) {
                const int64_t grow = (int64_t)rc * p.s + cur.zone_row0 + ro;
                p.lse[(int64_t)bh * p.S + grow] = (m_used + log2f(l)) * 0.6931471805599453f;
            }
        }
        if (rr == 0 && store_pending) tma_store_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 10) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"(TMEM_COLS) : "memory");
    }
    // the last CTA to leave puts the scheduler's counters back to zero for the next launch that uses them
    if (threadIdx.x == 0 && p.sched) {
        __threadfence();
        if (atomicAdd(p.sched + 1, 1u) == gridDim.x - 1) {
            p.sched[0] = 0;
            p.sched[1] = 0;
            __threadfence();
        }
    }
}

// ------------------------------------------------------------------ bounded-wait self test
// One thread waits on an mbarrier that nobody ever arrives on, with the same wait routine as the
// attention kernel but a limit of about a millisecond; it must give up, record LOMA_ERR_TIMEOUT in the
// status word and return, leaving the context usable.
__global__ void bounded_wait_selftest_kernel(int* status, long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const long long t0 = clock64();
    const uint32_t b = smem_u32(&bar);
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(b, 0)) return;            // cannot happen: no arrival is ever made
        if ((it & 63u) == 0 && clock64() - t0 > limit_cycles) {
            abort_flag = 1;
            atomicExch(status, (int)LOMA_ERR_TIMEOUT);
            return;
        }
    }
}

cudaError_t launch_bounded_wait_selftest(cudaStream_t st) {
    int* status = device_status_word();
    if (!status) return cudaErrorUnknown;
    bounded_wait_selftest_kernel<<<1, 1, 0, st>>>(status, 2000000ll);
    count_launches(1);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ host side
// Counters of the in-kernel scheduler: pairs of (next tile, CTAs finished), cleared by the last CTA of the
// launch that used them.  Two launches that may run at the same time must not share a pair, so a pair
// belongs to a stream (kernels of one stream never overlap): the first SCHED_STREAMS streams that call
// get one each.  A launch that is being captured into a CUDA graph may later be replayed on any stream,
// next to anything, so it gets a pair of its own that is never handed out again (SCHED_CAPTURES of them).
// When a table is full the launch runs without a counter: the kernel then deals the tiles round robin,
// which is a few percent slower on short layouts and just as correct.
constexpr int SCHED_STREAMS = 192, SCHED_CAPTURES = 320;
static __device__ unsigned g_sched_counters[SCHED_STREAMS + SCHED_CAPTURES][2];

static unsigned* sched_counters(cudaStream_t st) {
    static std::mutex mu;
    static unsigned* base[64] = {nullptr};
    static cudaStream_t owner[64][SCHED_STREAMS];
    static int n_owner[64] = {0}, n_capture[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!base[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_sched_counters) != cudaSuccess) return nullptr;
        base[dev] = static_cast<unsigned*>(ptr);
    }
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    if (cs != cudaStreamCaptureStatusNone) {
        if (n_capture[dev] >= SCHED_CAPTURES) return nullptr;
        return base[dev] + 2 * (SCHED_STREAMS + n_capture[dev]++);
    }
    for (int i = 0; i < n_owner[dev]; ++i)
        if (owner[dev][i] == st) return base[dev] + 2 * i;
    if (n_owner[dev] >= SCHED_STREAMS) return nullptr;
    owner[dev][n_owner[dev]] = st;
    return base[dev] + 2 * n_owner[dev]++;
}

// Launch of the kernel for a finished plan: per-device set-up (done once), grid size.
static cudaError_t launch_tc_kernel(const TmaMaps& maps, const FwdParams& p, int D, cudaStream_t st) {
    // SM count and the opt-in to large dynamic shared memory
    static int sm_count[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (sm_count[dev] == 0) {
        int sms = 0;
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(masked_attn_tc_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TcSmem<128>::TOTAL + 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(masked_attn_tc_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     TcSmem<128>::TOTAL + 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(masked_attn_tc_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     TcSmem<64>::TOTAL + 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(masked_attn_tc_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     TcSmem<64>::TOTAL + 1024);
        if (e != cudaSuccess) return e;
        sm_count[dev] = sms;
    }
    const int sms = sm_count[dev];
    const int64_t work = (int64_t)p.total_tiles * p.BH;
    const int64_t want = (work + 1) / 2;            // two streams (query tiles in flight) per CTA
    const int grid = (int)(want < sms ? want : sms);
    // the shared-memory footprint also keeps one CTA per SM (each allocates all 512 TMEM columns)
    const bool ragged = p.prefill && p.prefill_lens;
    if (D == 128) {
        if (ragged) masked_attn_tc_kernel<128, true><<<grid, TC_THREADS, TcSmem<128>::TOTAL + 1024, st>>>(maps, p);
        else masked_attn_tc_kernel<128, false><<<grid, TC_THREADS, TcSmem<128>::TOTAL + 1024, st>>>(maps, p);
    } else {
        if (ragged) masked_attn_tc_kernel<64, true><<<grid, TC_THREADS, TcSmem<64>::TOTAL + 1024, st>>>(maps, p);
        else masked_attn_tc_kernel<64, false><<<grid, TC_THREADS, TcSmem<64>::TOTAL + 1024, st>>>(maps, p);
    }
    count_launches(1);
    return cudaGetLastError();
}


struct MapCacheKey {
    const void *q, *k, *v, *o;
    int B, H, D, n, c, t, tail;
    unsigned flags;
    int64_t sb, sh, ss;
    bool operator==(const MapCacheKey& r) const {
        return q == r.q && k == r.k && v == r.v && o == r.o && B == r.B && H == r.H && D == r.D && n == r.n && c == r.c &&
               t == r.t && tail == r.tail && flags == r.flags && sb == r.sb && sh == r.sh && ss == r.ss;
    }
};

// Returns cudaErrorNotSupported when the tensor-core path cannot take the call
// (the caller then uses the CUDA-core kernel).
cudaError_t launch_masked_attn_tc(const void* q, const void* k, const void* v, void* o, float* lse, int B, int H, int D,
                                  const Layout& L, int64_t sb, int64_t sh, int64_t ss, float scale, cudaStream_t st) {
    if (!encode_fn()) return cudaErrorNotSupported;
    if (L.t > 256 * 128 || L.tc > (1 << 24)) return cudaErrorNotSupported;

    FwdParams p{};
    make_plan(L, B, H, &p);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.lse = lse;
    p.status = device_status_word();
    if (!p.status) return cudaErrorUnknown;
    if ((int64_t)p.total_tiles * p.BH > 0x7ffffff0ll - 2 * 148) return cudaErrorNotSupported;
    p.sched = sched_counters(st);   // NULL: static deal

    // tensor maps, cached for repeated calls on the same tensors with the same layout (the addresses are
    // part of the key only; nothing is read through them after the call)
    static std::mutex mu;
    static MapCacheKey cached_key{};
    static TmaMaps cached_maps;
    static bool have_cache = false;
    TmaMaps maps;
    {
        std::lock_guard<std::mutex> lock(mu);
        MapCacheKey key{q, k, v, o, B, H, D, L.n_chunks, L.c, L.t, L.tail_read, L.flags, sb, sh, ss};
        if (!(have_cache && key == cached_key)) {
            TmaMaps mnew{};
            const void* bases[4] = {q, k, v, o};
            CUtensorMap* arrs[4] = {mnew.q, mnew.k, mnew.v, mnew.o};
            for (int ti = 0; ti < 4; ++ti) {
                for (int vi = 0; vi < 4; ++vi) {
                    const View& vw = p.view[vi];
                    if (vw.ntiles == 0) continue;
                    const int64_t row0 = (vi == V_TAIL) ? (int64_t)L.n_chunks * L.s : vw.zone_row0;
                    if (!encode_view(&arrs[ti][vi], bases[ti], vw, D, B, H, row0, sb, sh, ss, L.s))
                        return cudaErrorNotSupported;
                }
            }
            cached_maps = mnew;
            cached_key = key;
            have_cache = true;
        }
        maps = cached_maps;
    }

    return launch_tc_kernel(maps, p, D, st);
}

// New tokens over an existing cache on the same kernel: the query view is the l new rows, the key view the
// cache rows 0 .. cache_len + l - 1 (the new rows' K/V have been appended before this launch).
// q, o: [B, H, l, D] contiguous; k_cache, v_cache: [B, H, cap, D] contiguous.  cache_lens (device, [B], or NULL): every
// sequence's own number of earlier entries; its tiles then stop at its own last key tile, whose rows past the
// sequence's end the caller has made finite (they are multiplied by probabilities of zero).
cudaError_t launch_prefill_attn_tc(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse, int B,
                                   int H, int D, int l, int cap, int cache_len, const int32_t* cache_lens,
                                   const Paging& pg, float scale, cudaStream_t st) {
    if (!encode_fn()) return cudaErrorNotSupported;
    if (pg.table && (!cache_lens || pg.log2_ps < 7)) return cudaErrorNotSupported;   // pages of a multiple of 128 rows
    FwdParams p{};
    make_prefill_plan(l, cache_len, B, H, &p);   // ragged batch: cache_len is the bound the per-sequence lengths are clamped to
    p.prefill_lens = cache_lens;
    p.page_table = pg.table; p.pt_stride = pg.max_pages; p.log2_ps = pg.log2_ps; p.n_pages = pg.n_pages;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.lse = lse;
    p.status = device_status_word();
    if (!p.status) return cudaErrorUnknown;
    if ((int64_t)p.total_tiles * p.BH > 0x7ffffff0ll - 2 * 148) return cudaErrorNotSupported;
    p.sched = sched_counters(st);   // NULL: static deal

    struct Key {
        const void *q, *k, *v, *o;
        int B, H, D, l, cap, cache_len, paged, log2_ps, n_pages;
        bool operator==(const Key& r) const {
            return q == r.q && k == r.k && v == r.v && o == r.o && B == r.B && H == r.H && D == r.D && l == r.l &&
                   cap == r.cap && cache_len == r.cache_len && paged == r.paged && log2_ps == r.log2_ps &&
                   n_pages == r.n_pages;
        }
    };
    static std::mutex mu;
    static Key cached_key{};
    static TmaMaps cached_maps;
    static bool have_cache = false;
    TmaMaps maps;
    {
        std::lock_guard<std::mutex> lock(mu);
        Key key{q, k_cache, v_cache, o, B, H, D, l, cap, cache_len, pg.table ? 1 : 0, pg.log2_ps, pg.n_pages};
        if (!(have_cache && key == cached_key)) {
            TmaMaps mnew{};
            const int64_t qs_h = (int64_t)l * D, qs_b = qs_h * H, cs_h = (int64_t)cap * D, cs_b = cs_h * H;
            const View& qv = p.view[V_TAIL];
            const View& kv = p.view[V_MEM];
            if (!encode_view(&mnew.q[V_TAIL], q, qv, D, B, H, 0, qs_b, qs_h, D, l) ||
                !encode_view(&mnew.o[V_TAIL], o, qv, D, B, H, 0, qs_b, qs_h, D, l))
                return cudaErrorNotSupported;
            if (pg.table) {
                // the pool [n_pages, H, page_size, D] seen as n_pages "batch elements" of one zone of page_size rows
                const int ps = 1 << pg.log2_ps;
                const View pv = make_view(ps, 1, 0, 0);
                const int64_t ps_h = (int64_t)ps * D, ps_b = ps_h * H;
                if (!encode_view(&mnew.k[V_MEM], k_cache, pv, D, pg.n_pages, H, 0, ps_b, ps_h, D, ps) ||
                    !encode_view(&mnew.v[V_MEM], v_cache, pv, D, pg.n_pages, H, 0, ps_b, ps_h, D, ps))
                    return cudaErrorNotSupported;
            } else if (!encode_view(&mnew.k[V_MEM], k_cache, kv, D, B, H, 0, cs_b, cs_h, D, cache_len + l) ||
                       !encode_view(&mnew.v[V_MEM], v_cache, kv, D, B, H, 0, cs_b, cs_h, D, cache_len + l)) {
                return cudaErrorNotSupported;
            }
            cached_maps = mnew;
            cached_key = key;
            have_cache = true;
        }
        maps = cached_maps;
    }
    return launch_tc_kernel(maps, p, D, st);
}

}  // namespace loma
