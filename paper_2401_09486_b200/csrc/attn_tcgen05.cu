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
// One persistent CTA (384 threads) per SM.  A CTA works on a PAIR of query tiles at a time (tiles 2i and
// 2i + 1 of one view and one (batch, head): A and B) and feeds both from one stream of key tiles -- two
// neighbouring tiles visit almost the same keys, so a K/V tile both need crosses into shared memory once
// (see "pairs of query tiles" in tile_plan.cuh for the merged order).  Shared memory: Q_A, Q_B, a two-stage
// ring of (K tile, V tile), and one 64-column output staging panel per tile.  TMEM: per tile a 128-column
// score region (the two 64-key halves of a key tile side by side) and a 128-column output accumulator.
//   warps 0-3 / 4-7   softmax warpgroup of tile A / B: thread = query row = TMEM lane.  The 128 keys of a
//                     step are taken as two halves of 64 ("events"): read the scores of a half, row maximum
//                     (three-input max), probabilities 2^(s*scale - ref) with packed two-wide fp32 FMA/ADD,
//                     bf16 P written back over the scores.  The output accumulates in TMEM; the reference
//                     maximum only moves, and the accumulator is only rescaled, when a row maximum has
//                     grown by more than 2^8.  Epilogue: normalise, round to bf16, stage 64 columns at a
//                     time, TMA store.
//   warp 8            TMA producer (one lane): draws the next pair, loads Q_A and Q_B, then K and V of every
//                     merged step into the ring; it runs ahead of the other roles as far as the ring and the
//                     Q buffers allow, across pair boundaries too.
//   warp 9 / 10       MMA issuer of tile A / B: control flow is warp-uniform and one elected lane issues.
//                     Per step: S = Q K^T with both operands in shared memory (N = 128 when both halves of
//                     the key tile are visited, N = 64 otherwise), then per visited half O += P_h V_h with P
//                     read from TMEM and V as an MN-major shared operand.  While one tile's warpgroup turns
//                     scores into probabilities the tensor pipe works for the other tile; a ring stage is
//                     refilled once both tiles (or the only one that visits the step) have released it.
// Pairs are handed out at run time from one counter over a statically ordered list (longest first,
// (batch, head) fastest).  Every mbarrier wait is bounded: on expiry the CTA records LOMA_ERR_TIMEOUT, all
// roles leave their loops, TMEM is freed and the kernel returns.
#include <type_traits>

#include "tcgen05_common.cuh"

namespace loma {

struct TmaMaps {
    CUtensorMap q[4], k[4], v[4], o[4];
};

// Optional clock counters of the roles' waits and a time line of the first CTA's events (compiled in with
// -DLOMA_KERNEL_TIMERS only; a development aid, read back with loma_debug_read_timers / _trace).
#ifdef LOMA_KERNEL_TIMERS
__device__ unsigned long long g_timers[160][48];
__device__ unsigned long long g_trace[8][4096];
#define TRACE(role, idx) do { if (blockIdx.x == 0 && (idx) < 4096) g_trace[role][idx] = (unsigned long long)clock64(); } while (0)
#define TIMER_DECL unsigned long long tmr_[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}; long long tmr_t0_ = 0; const long long tmr_begin_ = clock64()
#define TIMER_START() (tmr_t0_ = clock64())
#define TIMER_STOP(i) (tmr_[i] += (unsigned long long)(clock64() - tmr_t0_))
#define TIMER_COUNT(i) (++tmr_[i])
#define TIMER_FLUSH(base, n)                                                                    \
    do {                                                                                        \
        tmr_[(n) - 1] = (unsigned long long)(clock64() - tmr_begin_);                           \
        if (blockIdx.x < 160)                                                                   \
            for (int i_ = 0; i_ < (n); ++i_) g_timers[blockIdx.x][(base) + i_] += tmr_[i_];     \
    } while (0)
#else
#define TRACE(role, idx) ((void)0)
#define TIMER_DECL
#define TIMER_START() ((void)0)
#define TIMER_STOP(i) ((void)0)
#define TIMER_COUNT(i) ((void)0)
#define TIMER_FLUSH(base, n) ((void)0)
#endif

// ------------------------------------------------------------------ the kernel
constexpr int TC_THREADS = 384;   // 2 softmax warpgroups + 1 warpgroup holding the TMA warp and the two MMA warps
constexpr int TMEM_COLS = 512;

// mbarriers of a CTA
enum {
    B_QF = 0,    // +x   Q tile of A / B has landed
    B_QE = 2,    // +x   every score product of the pair's tile x has completed: Q buffer free
    B_KF = 4,    // +s   K tile of ring stage s has landed
    B_KE = 6,    // +s   every score product that reads stage s has completed (two arrivals: one per tile that visits the step, the missing one from the loader)
    B_VF = 8,    // +s
    B_VE = 10,   // +s   every P.V product that reads stage s has completed (two arrivals, as B_KE)
    B_SF = 12,   // +2x+(event & 1)   scores of an event of tile x are in TMEM
    B_PF = 16,   // +2x+(event & 1)   probabilities of an event are in TMEM (128 arrivals)
    B_OF = 20,   // +2x+(event & 1)   the P.V product of an event of tile x has completed
    B_TF = 24,   // +(n & 3)  the n-th pair number has been posted in slot n & 3 of the pair ring
    B_TE = 28,   // +(n & 3)  every reader (8 softmax warps, 2 MMA warps) has taken the n-th pair number
    NBAR = 32
};

// Shared memory: Q_A, Q_B, ring of two (K, V) stages, one output staging panel per tile.
template <int D>
struct TcSmem {
    static constexpr int PANELS = D / 64;
    static constexpr int PANEL_BYTES = 128 * 128;           // 128 rows x 64 bf16
    static constexpr int TILE_BYTES = PANELS * PANEL_BYTES; // one 128 x D tile
    static constexpr int Q_OFF = 0;                         // + x * TILE_BYTES
    static constexpr int K_OFF = 2 * TILE_BYTES;            // + s * 2 * TILE_BYTES
    static constexpr int V_OFF = 3 * TILE_BYTES;            // + s * 2 * TILE_BYTES
    static constexpr int O_OFF = 6 * TILE_BYTES;            // + x * PANEL_BYTES
    static constexpr int TOTAL = 6 * TILE_BYTES + 2 * PANEL_BYTES;
};

template <int D>
__global__ void __launch_bounds__(TC_THREADS, 1)
masked_attn_tc_kernel(const __grid_constant__ TmaMaps maps, const FwdParams p) {
    using SM = TcSmem<D>;
    constexpr int PANELS = SM::PANELS;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[NBAR];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int pair_ring_s[4];

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < NBAR; ++i)
            mbar_init(bar(i), (i >= B_PF && i < B_PF + 4) ? 128 : (i >= B_TE && i < B_TE + 4) ? 10
                                  : (i >= B_KE && i < B_KE + 2) || (i >= B_VE && i < B_VE + 2) ? 2 : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // zero the operand buffers once: rows a TMA box does not cover keep finite contents
    for (int i = threadIdx.x; i < SM::TOTAL / 16; i += TC_THREADS)
        reinterpret_cast<uint4*>(smem_gen)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem0 = tmem_slot;   // tile x: scores at tmem0 + 256 x, output accumulator at + 128
    volatile int* abortp = &abort_flag;

    // Pairs are handed out from one counter, longest first ((batch, head) fastest inside a rank).  The
    // producer draws the number and posts it in a four-slot ring (slot n & 3, barrier B_TF + (n & 3),
    // completion n >> 2, for the CTA's n-th pair); the MMA issuer and the warpgroups read it there and
    // acknowledge on B_TE, which the producer waits for before it reuses the slot (a warpgroup without a
    // tile in some pairs may lag behind the others).  A negative number ends the CTA's work.  Which CTA
    // computes a pair has no influence on the pair's result.  Without a counter (p.sched == NULL) the
    // pairs are dealt round robin.
    const int total_work = p.total_pairs * p.BH;
    volatile int* pair_ring = pair_ring_s;
    auto next_pair = [&](uint32_t n, bool& ok_) -> int {   // called by whole warps
        ok_ = __all_sync(0xffffffffu, mbar_wait(bar(B_TF + (n & 3)), (n >> 2) & 1, abortp, p.status));
        const int w = ok_ ? pair_ring[n & 3] : -1;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_TE + (n & 3)));
        return w;
    };

    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;" ::: "memory");
    }
    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t gl = 0, pcount = 0;      // K/V loads so far (one per merged step), pairs so far
            uint32_t nq[2] = {0, 0};          // uses of each Q buffer so far
            bool ok = true;
            TIMER_DECL;
            for (;; ++pcount) {
                int w = p.sched ? (int)atomicAdd(p.sched, 1u) : (int)(blockIdx.x + pcount * gridDim.x);
                if (w >= total_work || !ok) w = -1;
                if (pcount >= 4 && ok) ok = mbar_wait(bar(B_TE + (pcount & 3)), ((pcount >> 2) - 1) & 1, abortp, p.status);
                if (!ok) w = -1;
                pair_ring[pcount & 3] = w;
                __threadfence_block();
                mbar_arrive(bar(B_TF + (pcount & 3)));
                if (w < 0) break;
                const int rank = fdiv(w, p.dBH), bh = w - rank * p.BH;
                const int bi = fdiv(bh, p.dH), hi = bh - bi * p.H;
                PairDesc pd;
                decode_pair(p, rank, pd);
                const View& qv = p.view[pd.td[0].view];
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    if (x == 1 && !pd.nb) break;
                    TIMER_START();
                    if (nq[x] > 0) ok = mbar_wait(bar(B_QE + x), (nq[x] - 1) & 1, abortp, p.status);
                    TIMER_STOP(0);
                    if (!ok) break;
                    ++nq[x];
                    mbar_expect_tx(bar(B_QF + x), qv.R * qv.CH * 128 * PANELS);
                    for (int pn = 0; pn < PANELS; ++pn)
                        tma_load_5d(smem_base + SM::Q_OFF + x * SM::TILE_BYTES + pn * SM::PANEL_BYTES, &maps.q[pd.td[x].view],
                                    bar(B_QF + x), pn * 64, pd.td[x].r0, pd.td[x].c0, hi, bi);
                }
                if (!ok) break;
                for (int m = 0; m < pd.pm.nmerged; ++m, ++gl) {
                    int x, j;
                    merged_source(pd.pm, m, x, j);
                    KTile kt;
                    if (x) step_ktile(p, pd.td[1], j, kt);
                    else step_ktile(p, pd.td[0], j, kt);
                    const View& kv = p.view[kt.view];
                    const uint32_t s = gl & 1, ph = (gl >> 1) & 1;
                    const uint32_t bytes = kv.R * kv.CH * 128 * PANELS;
                    // a stage is released by two arrivals; where only one tile visits the step, the other one is given here
                    const bool lone = !visits_merged(pd.pm, 1 - x, m);
                    TIMER_START();
                    ok = mbar_wait(bar(B_KE + s), ph ^ 1, abortp, p.status);
                    TIMER_STOP(1);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_KF + s), bytes);
                    for (int pn = 0; pn < PANELS; ++pn)
                        tma_load_5d(smem_base + SM::K_OFF + s * 2 * SM::TILE_BYTES + pn * SM::PANEL_BYTES, &maps.k[kt.view],
                                    bar(B_KF + s), pn * 64, kt.r0, kt.c0, hi, bi);
                    if (lone) mbar_arrive(bar(B_KE + s));
                    TIMER_START();
                    ok = mbar_wait(bar(B_VE + s), ph ^ 1, abortp, p.status);
                    TIMER_STOP(2);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_VF + s), bytes);
                    for (int pn = 0; pn < PANELS; ++pn)
                        tma_load_5d(smem_base + SM::V_OFF + s * 2 * SM::TILE_BYTES + pn * SM::PANEL_BYTES, &maps.v[kt.view],
                                    bar(B_VF + s), pn * 64, kt.r0, kt.c0, hi, bi);
                    if (lone) mbar_arrive(bar(B_VE + s));
                }
                if (!ok) break;
            }
            TIMER_FLUSH(0, 4);
            if (!ok) {
                // leaving early (the abort flag is set): give copies in flight a bounded time to land
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000ll) {}
            }
        }
    } else if (warp == 9 || warp == 10) {
        // ------------------------------------------------------------ MMA issuer of tile X
        // All 32 lanes run the loops (warp-uniform); one elected lane issues the instructions.  One warp per
        // tile: an issuing thread runs in step with the tensor pipe (its queue is short), so the bookkeeping
        // between two instructions of one warp is covered by the other warp's instructions.
        const int X = warp - 9;
        // instruction descriptors: fp32 accumulate, bf16 x bf16, M = 128
        constexpr uint32_t IDESC_S64 = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
        constexpr uint32_t IDESC_PV =
            (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)D >> 3) << 17) | ((128u >> 4) << 24);
        const uint32_t tm = tmem0 + X * 256;
        const uint64_t qd = smem_desc(smem_base + SM::Q_OFF + X * SM::TILE_BYTES, 16, 1024);
        uint32_t ge = 0, gse = 0;         // events (visited halves) whose P.V / whose scores have been issued on this slot, all pairs
        uint32_t nq = 0;                  // pairs in which this slot was used
        uint32_t gbase = 0, pcount = 0;   // merged steps of earlier pairs, pairs so far
        bool ok = true;
        TIMER_DECL;
        for (;; ++pcount) {
            const int w = next_pair(pcount, ok);
            if (w < 0) break;
            const int rank = fdiv(w, p.dBH);
            PairMap pm;
            TileIssue ti;
            bool mine;
            {
                PairDesc pd;
                decode_pair(p, rank, pd);
                pm = pd.pm;
                mine = (X == 0) || pd.nb;
                if (mine) {
                    if (X) ti.start(pm, 1, tile_half_masks(p, pd.td[1], lane), pd.td[1].nsteps);
                    else ti.start(pm, 0, tile_half_masks(p, pd.td[0], lane), pd.td[0].nsteps);
                }
            }
            if (mine) {
                ++nq;
                IssueAct act;
                while (ok && !ti.done()) {
                    TIMER_START();
                    ti.next(act);
                    TIMER_STOP(4);
                    const uint32_t gl = gbase + (uint32_t)act.m, s = gl & 1, ph = (gl >> 1) & 1;
                    if (act.is_s) {
                        TIMER_START();
                        if (act.first_event)
                            ok = __all_sync(0xffffffffu, mbar_wait(bar(B_QF + X), (nq - 1) & 1, abortp, p.status));
                        if (ok && act.first_of_step) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_KF + s), ph, abortp, p.status));
                        TIMER_STOP(0);
                        if (!ok) break;
                        TIMER_START();
                        tc_fence_after();
                        if (elect_one()) {
                            const uint64_t kd = smem_desc(smem_base + SM::K_OFF + s * 2 * SM::TILE_BYTES, 16, 1024);
#pragma unroll
                            for (int kk = 0; kk < D / 16; ++kk) {
                                // descriptor start addresses are in 16-byte units; 64 key rows are 8192 bytes further
                                const uint64_t off = (uint64_t)(((kk >> 2) * SM::PANEL_BYTES + (kk & 3) * 32) >> 4);
                                mma_ss(tm + (gse & 1) * 64, qd + off, kd + off + (uint64_t)((act.h * 8192) >> 4), IDESC_S64, kk > 0);
                            }
                            tc_commit(bar(B_SF + 2 * X + (gse & 1)));
                            if (act.last_of_step) tc_commit(bar(B_KE + s));
                            if (act.last_s) tc_commit(bar(B_QE + X));
                        }
                        __syncwarp();
                        TIMER_STOP(5);
                        if (lane == 0) TRACE(4 * X + 2, gse);
                        ++gse;
                    } else {
                        TIMER_START();
                        ok = __all_sync(0xffffffffu, mbar_wait(bar(B_PF + 2 * X + (ge & 1)), (ge >> 1) & 1, abortp, p.status));
                        TIMER_STOP(1);
                        TIMER_START();
                        if (ok && act.first_of_step)
                            ok = __all_sync(0xffffffffu, mbar_wait(bar(B_VF + s), ph, abortp, p.status));
                        TIMER_STOP(2);
                        TIMER_COUNT(3);
                        if (!ok) break;
                        TIMER_START();
                        tc_fence_after();
                        if (elect_one()) {
                            const uint64_t vd = smem_desc(smem_base + SM::V_OFF + s * 2 * SM::TILE_BYTES, SM::PANEL_BYTES, 1024);
                            const int h = act.h;
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4)
                                mma_ts(tm + 128, tm + (ge & 1) * 64 + k4 * 8, vd + (uint64_t)(((h * 4 + k4) * 2048) >> 4), IDESC_PV,
                                       !act.first_event || (k4 > 0));
                            tc_commit(bar(B_OF + 2 * X + (ge & 1)));
                            if (act.last_of_step) tc_commit(bar(B_VE + s));
                        }
                        __syncwarp();
                        TIMER_STOP(6);
                        if (lane == 0) TRACE(4 * X + 3, ge);
                        ++ge;
                    }
                }
            }
            if (!ok) break;
            gbase += (uint32_t)pm.nmerged;
        }
        if (lane == 0) TIMER_FLUSH(8 + 8 * X, 8);
    } else if (warp < 8) {
        // ------------------------------------------------------------ softmax + epilogue of tile X (128 threads)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;" ::: "memory");
        const int X = warp >> 2;
        const int rr = threadIdx.x & 127;
        const uint32_t lane_addr = tmem0 + X * 256 + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t s_addr = lane_addr, o_addr = lane_addr + 128;
        const uint32_t o_stage = smem_base + SM::O_OFF + X * SM::PANEL_BYTES;
        uint8_t* o_stage_gen = smem_gen + SM::O_OFF + X * SM::PANEL_BYTES;
        uint32_t ge = 0;    // visited halves so far on this tile slot (see the MMA issuer)
        bool ok = true;
        bool store_pending = false;
        TIMER_DECL;
        // Everything this thread needs to know about a tile.  The next tile is decoded while the last
        // product of the current one drains, so the decode's chain of dependent loads and integer
        // arithmetic stays off the path between two tiles.
        struct TileCtx {
            TileDesc td;
            HalfMasks hm;
            int bh, bi, hi, ro, rc, zone_row0;
            bool row_valid;
        };
        // the pair's tile X, or false when the pair has no tile B
        auto decode_ctx = [&](int w, TileCtx& c) -> bool {
            const int rank = fdiv(w, p.dBH);
            c.bh = w - rank * p.BH;
            c.bi = fdiv(c.bh, p.dH);
            c.hi = c.bh - c.bi * p.H;
            int view, qa, nb;
            pair_tiles(p, rank, view, qa, nb);
            if (X == 1 && !nb) return false;
            decode_tile_at(p, view, qa + X, c.td);
            const View& qv = p.view[c.td.view];
            const int rsub = fdiv(rr, qv.dR);
            c.ro = c.td.r0 + (rr - rsub * qv.R);
            c.rc = c.td.a0 + rsub;
            c.zone_row0 = qv.zone_row0;
            c.row_valid = (rr < qv.R * qv.CH) && (c.rc <= c.td.a1) && (c.ro < qv.Z);
            c.hm = tile_half_masks(p, c.td, lane);
            return true;
        };
        // the next pair (from number n on) in which this warpgroup has a tile; -1 = no more
        uint32_t pcount = 0;
        auto next_ctx = [&](TileCtx& c) -> int {
            for (;;) {
                bool got = true;
                const int w = next_pair(pcount, got);
                if (!got) { ok = false; return -1; }
                if (w < 0) return -1;
                ++pcount;
                if (decode_ctx(w, c)) return w;
            }
        };
        TileCtx cur, nxt;
        int w_cur = next_ctx(cur), w_next = -1;
        for (; w_cur >= 0 && ok; w_cur = w_next, cur = nxt) {
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
                    row_interval(p.view[kt.view], kt, rc, ro, rr, row_valid, lo, hi2);
                }
                // One visited half of a key tile (64 keys) per pass, in score buffer ge & 1: the tensor
                // pipe works on the other buffer while this warpgroup works on this one.
                {
                    const int b = ge & 1;
                    TIMER_START();
                    ok = __all_sync(0xffffffffu, mbar_wait(bar(B_SF + 2 * X + b), (ge >> 1) & 1, abortp, p.status));
                    TIMER_STOP(0);
                    if (!ok) break;
                    if (rr == 0) TRACE(4 * X + 0, ge);
                    tc_fence_after();
                    const int lo_h = lo - 64 * hw.h;                  // allowed columns of this half: [lo_h, lo_h + span)
                    const uint32_t span = (uint32_t)(hi2 - lo);
                    const bool full = __all_sync(0xffffffffu, lo_h <= 0 && hi2 - 64 * hw.h >= 64);
                    const uint32_t sh_addr = s_addr + b * 64;
                    uint32_t s[64];
                    TIMER_START();
                    tmem_ld32(sh_addr, s);
                    tmem_ld32(sh_addr + 32, s + 32);
                    tmem_wait_ld();
                    if (!full) {
#pragma unroll
                        for (int e = 0; e < 64; ++e)
                            if ((uint32_t)(e - lo_h) >= span) s[e] = 0xff800000u;   // -inf: blocked for this row
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
                    TIMER_STOP(1);
                    if (!first && __any_sync(0xffffffffu, need)) {
                        TIMER_COUNT(6);
                        // rescale the accumulated output: wait until the previous event's P.V has landed in TMEM
                        ok = __all_sync(0xffffffffu, mbar_wait(bar(B_OF + 2 * X + ((ge - 1) & 1)), ((ge - 1) >> 1) & 1, abortp, p.status));
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
                    TIMER_START();
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
                    mbar_arrive(bar(B_PF + 2 * X + (ge & 1)));
                    TIMER_STOP(2);
                    if (rr == 0) TRACE(4 * X + 1, ge);
                }
            }
            TIMER_START();
            if (ok) w_next = next_ctx(nxt);
            TIMER_STOP(3);
            // the last P.V of the tile belongs to event ge - 1 (products complete in issue order)
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_OF + 2 * X + ((ge - 1) & 1)), ((ge - 1) >> 1) & 1, abortp, p.status));
            if (ok) tc_fence_after();
            TIMER_START();

            // epilogue: normalise, round to bf16, stage 64 output columns at a time in shared
            // memory, TMA store.  Every thread of the warpgroup reaches the first barrier for
            // every tile it started; it also makes giving up a uniform decision.
            const float inv = 1.f / l;
            uint8_t* orow = o_stage_gen + rr * 128;
            bool give_up = false;
#pragma unroll
            for (int pn = 0; pn < PANELS; ++pn) {
                if (rr == 0 && store_pending) tma_store_wait_read();   // the staging panel is free again
                if (pn == 0) {
                    uint32_t any_bad;
                    asm volatile(
                        "{\n.reg .pred p, q;\nsetp.ne.u32 p, %1, 0;\nbar.red.or.pred q, %2, 128, p;\nselp.u32 %0, 1, 0, q;\n}"
                        : "=r"(any_bad)
                        : "r"((uint32_t)(ok ? 0 : 1)), "r"(1 + X)
                        : "memory");
                    if (any_bad) { give_up = true; break; }
                } else {
                    asm volatile("bar.sync %0, 128;" ::"r"(1 + X) : "memory");
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t r[32];
                    tmem_ld32(o_addr + pn * 64 + c * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const int ci = c * 4 + q4;       // 16-byte chunk of the 128-byte panel row
                        uint4 u;
                        u.x = pack_bf16(__uint_as_float(r[q4 * 8 + 0]) * inv, __uint_as_float(r[q4 * 8 + 1]) * inv);
                        u.y = pack_bf16(__uint_as_float(r[q4 * 8 + 2]) * inv, __uint_as_float(r[q4 * 8 + 3]) * inv);
                        u.z = pack_bf16(__uint_as_float(r[q4 * 8 + 4]) * inv, __uint_as_float(r[q4 * 8 + 5]) * inv);
                        u.w = pack_bf16(__uint_as_float(r[q4 * 8 + 6]) * inv, __uint_as_float(r[q4 * 8 + 7]) * inv);
                        *reinterpret_cast<uint4*>(orow + ((ci ^ (rr & 7)) << 4)) = u;
                    }
                }
                fence_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(1 + X) : "memory");
                if (rr == 0) {
                    tma_store_5d(&maps.o[td.view], o_stage, pn * 64, td.r0, td.c0, hi, bi);
                    tma_store_commit();
                    store_pending = true;
                }
            }
            if (give_up) { ok = false; break; }
            TIMER_STOP(4);
            tc_fence_before();
            if (p.lse && row_valid) {
                const int64_t grow = (int64_t)rc * p.s + cur.zone_row0 + ro;
                p.lse[(int64_t)bh * p.S + grow] = (m_used + log2f(l)) * 0.6931471805599453f;
            }
        }
        if (rr == 0 && store_pending) tma_store_wait_all();
        if (rr == 0) TIMER_FLUSH(24 + 8 * X, 8);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
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

#ifdef LOMA_KERNEL_TIMERS
}  // namespace loma
// development aids: copy the counters to out[160*48] and clear them / copy the time line to out[8*4096]
extern "C" __attribute__((visibility("default"))) int loma_debug_read_timers(unsigned long long* out) {
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(out, loma::g_timers, sizeof(unsigned long long) * 160 * 48) != cudaSuccess) return -1;
    static unsigned long long zeros[160 * 48] = {0};
    return cudaMemcpyToSymbol(loma::g_timers, zeros, sizeof(zeros)) == cudaSuccess ? 0 : -1;
}
extern "C" __attribute__((visibility("default"))) int loma_debug_read_trace(unsigned long long* out) {
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    return cudaMemcpyFromSymbol(out, loma::g_trace, sizeof(unsigned long long) * 8 * 4096) == cudaSuccess ? 0 : -1;
}
namespace loma {
#endif

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
// Counters of the in-kernel scheduler: pairs of (next pair, CTAs finished), cleared by the last CTA of the
// launch that used them.  Two launches that may run at the same time must not share a pair, so a pair
// belongs to a stream (kernels of one stream never overlap): the first SCHED_STREAMS streams that call
// get one each.  A launch that is being captured into a CUDA graph may later be replayed on any stream,
// next to anything, so it gets a pair of its own that is never handed out again (SCHED_CAPTURES of them).
// When a table is full the launch runs without a counter: the kernel then deals the pairs round robin,
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
    if ((int64_t)p.total_pairs * p.BH > 0x7ffffff0ll - 2 * 148) return cudaErrorNotSupported;
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

    // per-device set-up, done once: SM count and the opt-in to large dynamic shared memory
    static int sm_count[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (sm_count[dev] == 0) {
        int sms = 0;
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(masked_attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TcSmem<128>::TOTAL + 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(masked_attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 TcSmem<64>::TOTAL + 1024);
        if (e != cudaSuccess) return e;
        sm_count[dev] = sms;
    }
    const int sms = sm_count[dev];
    const int64_t work = (int64_t)p.total_pairs * p.BH;
    const int grid = (int)(work < sms ? work : sms);
    // the shared-memory footprint also keeps one CTA per SM (each allocates all 512 TMEM columns)
    if (D == 128)
        masked_attn_tc_kernel<128><<<grid, TC_THREADS, TcSmem<128>::TOTAL + 1024, st>>>(maps, p);
    else
        masked_attn_tc_kernel<64><<<grid, TC_THREADS, TcSmem<64>::TOTAL + 1024, st>>>(maps, p);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace loma
