// Tile plan of the tensor-core masked forward: how the laid-out sequence is cut
// into 128-row tiles of the four zone views, which key tiles each query tile
// visits, and which columns of a visited tile a row may attend to (Eq. 1-3).
// Plain integer logic shared by the kernel (device) and by the host-side
// reconstruction of the mask that the tests compare with the oracle's.
#pragma once

#include "loma_internal.cuh"

namespace loma {

__host__ __device__ __forceinline__ int plan_min(int a, int b) { return a < b ? a : b; }
__host__ __device__ __forceinline__ int plan_max(int a, int b) { return a > b ? a : b; }

// Division by a divisor fixed at launch, as one multiply-high, one subtract, one add and two shifts
// (Granlund and Montgomery, "Division by invariant integers using multiplication", 1994, the
// unsigned 32-bit case); exact for every numerator 0 <= n < 2^32.  The kernel decodes a tile with
// half a dozen dependent divisions, which as emulated hardware divisions cost over a microsecond.
struct FastDiv {
    unsigned mul, sh1, sh2;
};
inline FastDiv make_fastdiv(int d) {
    if (d < 1) d = 1;
    int l = 0;
    while ((1ull << l) < (unsigned long long)d) ++l;
    FastDiv f;
    f.mul = (unsigned)((((1ull << l) - (unsigned long long)d) << 32) / (unsigned long long)d + 1ull);
    f.sh1 = l < 1 ? l : 1;
    f.sh2 = l > 1 ? l - 1 : 0;
    return f;
}
__host__ __device__ __forceinline__ int fdiv(int n, const FastDiv& f) {
#ifdef __CUDA_ARCH__
    const unsigned t = __umulhi(f.mul, (unsigned)n);
#else
    const unsigned t = (unsigned)(((unsigned long long)f.mul * (unsigned)n) >> 32);
#endif
    return (int)((t + (((unsigned)n - t) >> f.sh1)) >> f.sh2);
}

enum { V_READ = 0, V_MEM = 1, V_REP = 2, V_TAIL = 3 };
enum { M_LT = 0, M_LE = 1, M_EQ = 2, M_CAUSAL = 3, M_DIAG = 4, M_CAUSAL_OFF = 5 };   // M_CAUSAL_OFF: causal with the diagonal moved by View::diag

struct View {
    int Z;           // zone length (rows per chunk in this view)
    int R;           // rows of one chunk inside a tile: min(Z, 128)
    int CH;          // chunks per tile: 1 if Z >= 128 else 128 / Z
    int tpc;         // tiles per chunk (Z >= 128) else 0
    int ntiles;      // tiles in the view
    int nch;         // chunks in the view
    int chunk_base;  // absolute chunk number of the view's chunk 0 (n_chunks for the tail)
    int zone_row0;   // first row of the zone inside its chunk
    int diag;        // key views of the prefill plan: row o of the query view sees keys 0 .. o + diag (M_CAUSAL_OFF)
    FastDiv dR, dCH, dtpc;   // division by R, CH and tpc
};

struct FwdParams {
    View view[4];
    int n_chunks, s, S, H, BH;
    int total_tiles;
    int n_tail, n_read, n_mem, n_rep;   // tiles per view, in scheduling order
    unsigned flags;
    int prefill;       // 1: the plan of loma_prefill_attn (query view V_TAIL over the new tokens, key view V_MEM over the cache)
    const int* prefill_lens;   // prefill plan of a ragged batch: [B] cache lengths on the device (NULL: uniform)
    const int* page_table;     // ... over a paged cache: block table [B, pt_stride] (pages of 2^log2_ps >= 128 rows)
    int pt_stride, log2_ps, n_pages;
    FastDiv dBH, dH, dTT;   // division by BH, H and total_tiles
    float scale_log2;
    float* lse;
    int* status;
    unsigned* sched;   // [0] next tile to hand out, [1] CTAs that have finished (the last one clears both); NULL = static deal
};

// Work item w of a launch -> tile rank and (batch, head): the tiles of one (b,h) are handed out together,
// longest first, before the next pair's.  The streams of the whole GPU then work on one or two pairs at a
// time, whose K and V (35 MB per head on the 69632-token layout, 4.4 MB per pair for a prompt piece over
// 8192 cache rows) stay in L2 while every tile of the pair streams them: each row is fetched from HBM once.
// (Handing out one rank for every (b,h) before the next rank -- longest tiles first over the whole launch --
// kept all pairs in flight at once: the prompt piece then read its cache four times and was bound by that,
// 2.82 ms against 2.22 ms, and the 69632-token layout took 1.40 ms against 1.32 ms.)
__host__ __device__ __forceinline__ void split_work(const FwdParams& p, int w, int& rank, int& bh) {
    bh = fdiv(w, p.dTT);
    rank = w - bh * p.total_tiles;
}


struct Seg {
    int view, mode, first, count;
};
struct TileDesc {
    int view, qi, c0, r0;   // view, tile index, first chunk (view-relative), first row in zone
    int a0, a1;             // absolute first / last chunk covered
    Seg seg[2];
    int nsteps;
};
struct KTile {
    int view, mode, c0, r0, a0;   // view-relative chunk, first row, absolute chunk
};

// ------------------------------------------------------------------ tile lists
__host__ __device__ __forceinline__ int tile_of_chunk(const View& v, int c) { return v.Z >= 128 ? c * v.tpc : fdiv(c, v.dCH); }
__host__ __device__ __forceinline__ int tiles_covering(const View& v, int nchunks) {
    return v.Z >= 128 ? nchunks * v.tpc : fdiv(nchunks + v.CH - 1, v.dCH);
}

// own_diag >= 0: the prefill plan of a ragged batch, where every sequence has its own cache length (at most the key
// view's diag, for which the plan was sized)
__host__ __device__ __forceinline__ void decode_tile(const FwdParams& p, int rank, TileDesc& td, int own_diag = -1) {
    int view, qi;
    if (rank < p.n_tail) { view = V_TAIL; qi = p.n_tail - 1 - rank; }
    else if ((rank -= p.n_tail) < p.n_read) { view = V_READ; qi = p.n_read - 1 - rank; }
    else if ((rank -= p.n_read) < p.n_mem) { view = V_MEM; qi = p.n_mem - 1 - rank; }
    else { view = V_REP; qi = rank - p.n_mem; }
    const View& g = p.view[view];
    td.view = view; td.qi = qi;
    int c1;
    if (g.Z >= 128) { td.c0 = fdiv(qi, g.dtpc); td.r0 = (qi - td.c0 * g.tpc) * 128; c1 = td.c0; }
    else { td.c0 = qi * g.CH; td.r0 = 0; c1 = plan_min(td.c0 + g.CH, g.nch) - 1; }
    td.a0 = g.chunk_base + td.c0;
    td.a1 = g.chunk_base + c1;
    const View& vm = p.view[V_MEM];
    const View& vr = p.view[V_READ];
    const int sub = (g.Z >= 128) ? qi - td.c0 * g.tpc : 0;   // tile index inside its chunk
    if (p.prefill) {
        // new tokens over the cache (Appendix A, inference_input): key tiles 0 .. the one that holds the
        // diagonal of the tile's last row (row o sees keys 0 .. o + diag)
        const int last_row = plan_min(td.r0 + 127, g.Z - 1);
        td.seg[0] = Seg{V_MEM, M_CAUSAL_OFF, 0, (last_row + (own_diag >= 0 ? own_diag : vm.diag)) / 128 + 1};
        td.seg[1] = Seg{V_MEM, M_CAUSAL_OFF, 0, 0};
    } else if (view == V_READ || view == V_TAIL) {
        // memory zones of every earlier chunk, then the own reading zone up to this tile
        td.seg[0] = Seg{V_MEM, M_LT, 0, tiles_covering(vm, td.a1)};
        td.seg[1] = Seg{view, M_CAUSAL, (g.Z >= 128) ? td.c0 * g.tpc : qi, sub + 1};
    } else if (view == V_MEM) {
        if (p.flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM)
            td.seg[0] = Seg{V_MEM, M_LE, 0, (g.Z >= 128) ? (td.a0 + 1) * g.tpc : qi + 1};
        else
            td.seg[0] = Seg{V_MEM, M_EQ, (g.Z >= 128) ? td.c0 * g.tpc : qi, (g.Z >= 128) ? g.tpc : 1};
        const int f = tile_of_chunk(vr, td.a0);
        td.seg[1] = Seg{V_READ, M_EQ, f, (vr.Z >= 128) ? (td.a1 - td.a0 + 1) * vr.tpc : tile_of_chunk(vr, td.a1) - f + 1};
    } else {
        const int f = tile_of_chunk(vm, td.a0);
        td.seg[0] = Seg{V_MEM, M_EQ, f, (vm.Z >= 128) ? (td.a1 - td.a0 + 1) * vm.tpc : tile_of_chunk(vm, td.a1) - f + 1};
        td.seg[1] = Seg{V_REP, M_DIAG, qi, 1};
    }
    td.nsteps = td.seg[0].count + td.seg[1].count;
}

__host__ __device__ __forceinline__ void step_ktile(const FwdParams& p, const TileDesc& td, int j, KTile& kt) {
    const bool first = j < td.seg[0].count;
    const int view = first ? td.seg[0].view : td.seg[1].view;
    const int mode = first ? td.seg[0].mode : td.seg[1].mode;
    const int t = first ? td.seg[0].first + j : td.seg[1].first + (j - td.seg[0].count);
    const View& g = p.view[view];
    kt.view = view; kt.mode = mode;
    if (g.Z >= 128) { kt.c0 = fdiv(t, g.dtpc); kt.r0 = (t - kt.c0 * g.tpc) * 128; }
    else { kt.c0 = t * g.CH; kt.r0 = 0; }
    kt.a0 = g.chunk_base + kt.c0;
}

// Allowed columns [lo, hi) of a key tile for a row at (chunk rc, offset ro), tile-local row rr.
// diag (mode M_CAUSAL_OFF only): the key view's diag, or the sequence's own cache length in a ragged batch.
__host__ __device__ __forceinline__ void row_interval(const View& kv, const KTile& kt, int rc, int ro, int rr, bool row_valid,
                                             int& lo, int& hi, int diag) {
    const int vcols = plan_min(kv.R, kv.Z - kt.r0);   // valid columns per chunk of this tile
    const int d = rc - kt.a0;
    lo = 0; hi = 0;
    if (kt.mode == M_LT || kt.mode == M_LE) {
        const int nch = plan_min(plan_max(d + (kt.mode == M_LE ? 1 : 0), 0), kv.CH);
        hi = nch > 0 ? (nch - 1) * kv.R + vcols : 0;
    } else if (kt.mode == M_DIAG) {
        lo = rr; hi = rr + 1;
    } else if (kt.mode == M_CAUSAL_OFF) {
        hi = plan_min(plan_max(ro + diag - kt.r0 + 1, 0), vcols);
    } else if (d >= 0 && d < kv.CH) {
        lo = d * kv.R;
        hi = lo + (kt.mode == M_EQ ? vcols : plan_min(plan_max(ro - kt.r0 + 1, 0), vcols));
    }
    if (!row_valid) { lo = 0; hi = 0; }
}

// Halves (64 columns each) of a key tile that hold an allowed column for at least one row of the
// query tile: bit h set = columns [64h, 64h + 64) are visited.  Computed from the union of the row
// intervals over the tile's chunks; a superset is harmless (every row still applies its own
// interval), a missing half would drop allowed entries, which the host-side coverage replay checks.
__host__ __device__ __forceinline__ unsigned step_halves(const FwdParams& p, const TileDesc& td, const KTile& kt, int own_diag = -1) {
    const View& kv = p.view[kt.view];
    const int vcols = plan_min(kv.R, kv.Z - kt.r0);
    int ulo = 0, uhi = 0;
    if (kt.mode == M_LT || kt.mode == M_LE) {
        const int nch = plan_min(plan_max(td.a1 - kt.a0 + (kt.mode == M_LE ? 1 : 0), 0), kv.CH);
        uhi = nch > 0 ? (nch - 1) * kv.R + vcols : 0;
    } else if (kt.mode == M_DIAG) {
        uhi = 128;
    } else if (kt.mode == M_CAUSAL_OFF) {
        const int last_row = plan_min(td.r0 + 127, p.view[td.view].Z - 1);
        uhi = plan_min(plan_max(last_row + (own_diag >= 0 ? own_diag : kv.diag) - kt.r0 + 1, 0), vcols);
    } else {
        const int d0 = plan_max(td.a0 - kt.a0, 0), d1 = plan_min(td.a1 - kt.a0, kv.CH - 1);
        if (d1 >= d0) { ulo = d0 * kv.R; uhi = d1 * kv.R + vcols; }
    }
    const unsigned m = ((ulo < 64 && uhi > 0) ? 1u : 0u) | (uhi > 64 ? 2u : 0u);
    return m ? m : 1u;
}

// Visited halves of a tile's steps as two bit masks: bit j of m[h] = half h of step j is visited.
// Steps from 64 on are taken whole, so that two 64-bit words always suffice.
struct HalfMasks {
    unsigned long long m[2];
    // visited halves of step j as two bits (bit h = half h)
    __host__ __device__ __forceinline__ unsigned bits(int j) const {
        return j >= 64 ? 3u : (unsigned)((m[0] >> j) & 1ull) | ((unsigned)((m[1] >> j) & 1ull) << 1);
    }
};
__host__ __device__ __forceinline__ unsigned visited_halves(const FwdParams& p, const TileDesc& td, int j, int own_diag = -1) {
    if (j >= 64) return 3u;
    KTile kt;
    step_ktile(p, td, j, kt);
    return step_halves(p, td, kt, own_diag);
}

// Walks the visited halves of a query tile's key tiles in order.  One visited half ("event") is
// the unit of the kernel's pipeline: one score buffer, one softmax pass, one P.V product.
struct HalfWalk {
    int j, h;
    unsigned cur;   // visited halves of step j (looked up once per step)
    __host__ __device__ __forceinline__ void start(const HalfMasks& hm) { j = 0; cur = hm.bits(0); h = (cur & 1u) ? 0 : 1; }
    __host__ __device__ __forceinline__ bool done(int nsteps) const { return j >= nsteps; }
    __host__ __device__ __forceinline__ void next(const HalfMasks& hm) {
        if (h == 0 && (cur & 2u)) { h = 1; return; }
        ++j;
        cur = hm.bits(j);
        h = (cur & 1u) ? 0 : 1;
    }
    __host__ __device__ __forceinline__ bool first_of_step(const HalfMasks&) const { return h == 0 || !(cur & 1u); }
    __host__ __device__ __forceinline__ bool last_of_step(const HalfMasks&) const { return h == 1 || !(cur & 2u); }
};

// ------------------------------------------------------------------ the plan read by key tile
// The backward's dK/dV pass owns one key tile at a time and walks the query tiles that visit it:
// the lists of decode_tile turned round.  A key tile of a view has the geometry of the query tile
// with the same index; the query tiles that visit it form at most four runs of consecutive tiles,
// one per view.  The host replays this side too and compares it with Eq. 2.
struct KeyTileDesc {
    int view, ki, c0, r0, a0, a1;
    Seg seg[4];
    int nseg, nsteps;
};
struct QTile {
    int view, mode, c0, r0, a0, a1;
};

__host__ __device__ __forceinline__ int last_tile_of_chunk(const View& v, int c) {
    return v.Z >= 128 ? (c + 1) * v.tpc - 1 : fdiv(c, v.dCH);
}

__host__ __device__ __forceinline__ void tile_geometry(const View& g, int ti, int& c0, int& r0, int& a0, int& a1) {
    int c1;
    if (g.Z >= 128) { c0 = fdiv(ti, g.dtpc); r0 = (ti - c0 * g.tpc) * 128; c1 = c0; }
    else { c0 = ti * g.CH; r0 = 0; c1 = plan_min(c0 + g.CH, g.nch) - 1; }
    a0 = g.chunk_base + c0;
    a1 = g.chunk_base + c1;
}

// Key tiles in scheduling order: memory tiles first (tile 0 is visited by the most query tiles),
// then the tail, reading and repetition tiles.
__host__ __device__ __forceinline__ void decode_key_tile(const FwdParams& p, int rank, KeyTileDesc& kd) {
    int view, ki;
    if (rank < p.n_mem) { view = V_MEM; ki = rank; }
    else if ((rank -= p.n_mem) < p.n_tail) { view = V_TAIL; ki = rank; }
    else if ((rank -= p.n_tail) < p.n_read) { view = V_READ; ki = rank; }
    else { view = V_REP; ki = rank - p.n_read; }
    const View& g = p.view[view];
    kd.view = view; kd.ki = ki;
    tile_geometry(g, ki, kd.c0, kd.r0, kd.a0, kd.a1);
    const View& vm = p.view[V_MEM];
    const View& vr = p.view[V_READ];
    const View& vp = p.view[V_REP];
    // four fixed slots (an absent run has count 0), written with compile-time indices so that they stay in registers
    const Seg none = Seg{view, M_EQ, 0, 0};
    kd.seg[0] = kd.seg[1] = kd.seg[2] = kd.seg[3] = none;
    auto run = [](int v, int mode, int first, int count) { return Seg{v, mode, first, count > 0 ? count : 0}; };
    if (view == V_MEM) {
        // reading rows of every later chunk and of the tail (Eq. 3)
        if (kd.a0 + 1 < p.n_chunks) { const int f = tile_of_chunk(vr, kd.a0 + 1); kd.seg[0] = run(V_READ, M_LT, f, p.n_read - f); }
        kd.seg[1] = run(V_TAIL, M_LT, 0, p.n_tail);
        // memory rows: own chunk (Eq. 1, row 2); with the prior-memory flag every later chunk too
        const int f = (g.Z >= 128) ? kd.c0 * g.tpc : ki;
        if (p.flags & LOMA_FLAG_MEM_SEES_PRIOR_MEM) kd.seg[2] = run(V_MEM, M_LE, f, p.n_mem - f);
        else kd.seg[2] = run(V_MEM, M_EQ, f, (g.Z >= 128) ? g.tpc : 1);
        // repetition rows of the same chunks (Eq. 1, row 3)
        if (p.n_rep > 0) { const int fr = tile_of_chunk(vp, kd.a0); kd.seg[3] = run(V_REP, M_EQ, fr, last_tile_of_chunk(vp, kd.a1) - fr + 1); }
    } else if (view == V_READ) {
        kd.seg[0] = run(V_READ, M_CAUSAL, ki, (g.Z >= 128) ? (kd.c0 + 1) * g.tpc - ki : 1);
        const int fm = tile_of_chunk(vm, kd.a0);
        kd.seg[1] = run(V_MEM, M_EQ, fm, last_tile_of_chunk(vm, kd.a1) - fm + 1);
    } else if (view == V_TAIL) {
        kd.seg[0] = run(V_TAIL, M_CAUSAL, ki, p.n_tail - ki);
    } else {
        kd.seg[0] = run(V_REP, M_DIAG, ki, 1);
    }
    kd.nseg = 4;
    kd.nsteps = kd.seg[0].count + kd.seg[1].count + kd.seg[2].count + kd.seg[3].count;
}

__host__ __device__ __forceinline__ void step_qtile(const FwdParams& p, const KeyTileDesc& kd, int j, QTile& qt) {
    // the run that holds step j (compile-time indices; runs with count 0 are stepped over)
    Seg sg = kd.seg[0];
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        if (j >= sg.count) {
            j -= sg.count;
            sg = kd.seg[i + 1];
        }
    }
    qt.view = sg.view; qt.mode = sg.mode;
    tile_geometry(p.view[qt.view], sg.first + j, qt.c0, qt.r0, qt.a0, qt.a1);
}

// Rows of a query tile that hold a row of the sequence: always a prefix [0, n).
__host__ __device__ __forceinline__ int valid_tile_rows(const View& g, int r0, int a0, int a1) {
    return g.Z >= 128 ? plan_min(128, g.Z - r0) : (a1 - a0 + 1) * g.R;
}

// Query rows [lo, hi) of query tile qt that may attend to the key at (chunk kc, offset ko), tile-local key row kr:
// row_interval read by column.
__host__ __device__ __forceinline__ void col_interval(const View& qv, const QTile& qt, int kc, int ko, int kr, bool key_valid,
                                                      int& lo, int& hi) {
    const int nvalid = valid_tile_rows(qv, qt.r0, qt.a0, qt.a1);
    const int vrows = plan_min(qv.R, qv.Z - qt.r0);   // valid rows per chunk of this tile
    const int d = kc - qt.a0;                         // the key's chunk relative to the tile's first chunk
    lo = 0; hi = 0;
    if (qt.mode == M_LT || qt.mode == M_LE) {
        const int first = plan_max(d + (qt.mode == M_LT ? 1 : 0), 0);   // first chunk of the tile that sees the key
        lo = first * qv.R; hi = nvalid;
    } else if (qt.mode == M_DIAG) {
        lo = kr; hi = kr + 1;
    } else if (d >= 0 && d < qv.CH) {
        lo = d * qv.R + (qt.mode == M_CAUSAL ? plan_min(plan_max(ko - qt.r0, 0), vrows) : 0);
        hi = d * qv.R + vrows;
    }
    if (hi > nvalid) hi = nvalid;
    if (!key_valid || hi < lo) { lo = 0; hi = 0; }
}

// Halves (64 query rows each) of step j that some key row of the tile may be seen from.
__host__ __device__ __forceinline__ unsigned visited_qhalves(const FwdParams& p, const KeyTileDesc& kd, int j) {
    if (j >= 64) return 3u;
    QTile qt;
    step_qtile(p, kd, j, qt);
    const View& qv = p.view[qt.view];
    const int nvalid = valid_tile_rows(qv, qt.r0, qt.a0, qt.a1);
    int ulo = 0, uhi = nvalid;
    if (qt.mode == M_LT || qt.mode == M_LE) {
        ulo = plan_max(kd.a0 - qt.a0 + (qt.mode == M_LT ? 1 : 0), 0) * qv.R;
    } else if (qt.mode != M_DIAG) {
        const int d0 = plan_max(kd.a0 - qt.a0, 0), d1 = plan_min(kd.a1 - qt.a0, qv.CH - 1);
        if (d1 >= d0) { ulo = d0 * qv.R; uhi = plan_min(nvalid, (d1 + 1) * qv.R); } else { uhi = 0; }
    }
    const unsigned m = ((ulo < 64 && uhi > 0) ? 1u : 0u) | (uhi > 64 ? 2u : 0u);
    return m ? m : 1u;
}

// Fills the geometry part of FwdParams (views, tile counts) from the layout.
inline View make_view(int Z, int nch, int chunk_base, int zone_row0) {
    View v{};
    v.Z = Z; v.nch = nch; v.chunk_base = chunk_base; v.zone_row0 = zone_row0;
    v.dR = v.dCH = v.dtpc = make_fastdiv(1);
    if (Z <= 0 || nch <= 0) { v.R = 1; v.CH = 1; v.tpc = 0; v.ntiles = 0; v.Z = (Z > 0 ? Z : 1); v.nch = 0; return v; }
    v.R = Z < 128 ? Z : 128;
    v.CH = Z >= 128 ? 1 : 128 / Z;
    v.tpc = Z >= 128 ? (Z + 127) / 128 : 0;
    v.ntiles = Z >= 128 ? nch * v.tpc : (nch + v.CH - 1) / v.CH;
    v.dR = make_fastdiv(v.R); v.dCH = make_fastdiv(v.CH); v.dtpc = make_fastdiv(v.tpc);
    return v;
}

inline void make_plan(const Layout& L, int B, int H, FwdParams* p) {
    p->view[V_READ] = make_view(L.tc, L.n_chunks, 0, 0);
    p->view[V_MEM] = make_view(L.t, L.n_chunks, 0, L.tc);
    p->view[V_REP] = make_view(L.tc, (L.flags & LOMA_FLAG_NO_REP_ZONE) ? 0 : L.n_chunks, 0, L.tc + L.t);
    p->view[V_TAIL] = make_view(L.tail_read, L.tail_read > 0 ? 1 : 0, L.n_chunks, 0);
    p->n_chunks = L.n_chunks; p->s = L.s; p->S = L.S; p->H = H; p->BH = B * H;
    p->n_tail = p->view[V_TAIL].ntiles; p->n_read = p->view[V_READ].ntiles;
    p->n_mem = p->view[V_MEM].ntiles; p->n_rep = p->view[V_REP].ntiles;
    p->total_tiles = p->n_tail + p->n_read + p->n_mem + p->n_rep;
    p->flags = L.flags; p->prefill = 0; p->prefill_lens = nullptr; p->page_table = nullptr;
    p->dBH = make_fastdiv(p->BH); p->dH = make_fastdiv(H); p->dTT = make_fastdiv(p->total_tiles);
}

// The plan of loma_prefill_attn: l new tokens (query view V_TAIL, one "chunk" of l rows) over a cache that holds
// cache_len earlier entries followed by the l new ones (key view V_MEM, one chunk of cache_len + l rows); row o
// sees keys 0 .. o + cache_len.
inline void make_prefill_plan(int l, int cache_len, int B, int H, FwdParams* p) {
    p->view[V_READ] = make_view(0, 0, 0, 0);
    p->view[V_MEM] = make_view(cache_len + l, 1, 0, 0);
    p->view[V_MEM].diag = cache_len;
    p->view[V_REP] = make_view(0, 0, 0, 0);
    p->view[V_TAIL] = make_view(l, 1, 0, 0);
    p->n_chunks = 0; p->s = 0; p->S = l; p->H = H; p->BH = B * H;
    p->n_tail = p->view[V_TAIL].ntiles; p->n_read = 0; p->n_mem = 0; p->n_rep = 0;
    p->total_tiles = p->n_tail;
    p->flags = 0; p->prefill = 1; p->prefill_lens = nullptr; p->page_table = nullptr;
    p->dBH = make_fastdiv(p->BH); p->dH = make_fastdiv(H); p->dTT = make_fastdiv(p->total_tiles);
}

}  // namespace loma
