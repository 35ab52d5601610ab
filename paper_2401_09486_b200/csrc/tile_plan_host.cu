// Host-side replay of the tensor-core kernel's tile plan.
#include <string.h>

#include "tile_plan.cuh"

namespace loma {

// counts[i*S + j] = number of (query tile, key tile) visits in which row i
// attends to column j.  A correct plan gives exactly the 0/1 mask of Eq. 2.
void plan_coverage_host(const Layout& L, uint8_t* counts) {
    FwdParams p{};
    make_plan(L, 1, 1, &p);
    memset(counts, 0, (size_t)L.S * L.S);
    for (int rank = 0; rank < p.total_tiles; ++rank) {
        TileDesc td;
        decode_tile(p, rank, td);
        const View& qv = p.view[td.view];
        // the same walk over visited halves as the kernel's roles take
        HalfMasks hm{{0, 0}};
        for (int j = 0; j < td.nsteps && j < 64; ++j) {
            const unsigned v = visited_halves(p, td, j);
            hm.m[0] |= (unsigned long long)(v & 1u) << j;
            hm.m[1] |= (unsigned long long)((v >> 1) & 1u) << j;
        }
        HalfWalk hw;
        for (hw.start(hm); !hw.done(td.nsteps); hw.next(hm)) {
            KTile kt;
            step_ktile(p, td, hw.j, kt);
            const View& kv = p.view[kt.view];
            for (int rr = 0; rr < 128; ++rr) {
                const int rsub = rr / qv.R;
                const int ro = td.r0 + (rr - rsub * qv.R);
                const int rc = td.a0 + rsub;
                const bool row_valid = (rr < qv.R * qv.CH) && (rc <= td.a1) && (ro < qv.Z);
                int lo, hi;
                row_interval(kv, kt, rc, ro, rr, row_valid, lo, hi, kv.diag);
                if (!row_valid || hi <= lo) continue;
                const int64_t grow = (int64_t)rc * L.s + qv.zone_row0 + ro;
                for (int col = (lo > 64 * hw.h ? lo : 64 * hw.h); col < hi && col < 64 * hw.h + 64; ++col) {
                    // column of the key tile -> row of the laid-out sequence, the way the TMA box gathers it
                    const int ksub = col / kv.R;
                    const int ko = kt.r0 + (col - ksub * kv.R);
                    const int kc = kt.a0 + ksub;
                    const int64_t gcol = (int64_t)kc * L.s + kv.zone_row0 + ko;
                    if (grow < L.S && gcol >= 0 && gcol < L.S) {
                        uint8_t& c = counts[grow * L.S + gcol];
                        if (c < 255) ++c;
                    }
                }
            }
        }
    }
}

// The plan of loma_prefill_attn replayed the same way: counts[i * (cache_len + l) + j] = visits in which new
// token i attends to key j (cached entries 0 .. cache_len - 1, then the new tokens).  A correct plan gives
// tril(ones(l, l + cache_len), diagonal = cache_len).
void prefill_plan_coverage_host(int l, int cache_len, uint8_t* counts) {
    FwdParams p{};
    make_prefill_plan(l, cache_len, 1, 1, &p);
    const int64_t W = (int64_t)cache_len + l;
    memset(counts, 0, (size_t)l * W);
    for (int rank = 0; rank < p.total_tiles; ++rank) {
        TileDesc td;
        decode_tile(p, rank, td);
        const View& qv = p.view[td.view];
        HalfMasks hm{{0, 0}};
        for (int j = 0; j < td.nsteps && j < 64; ++j) {
            const unsigned v = visited_halves(p, td, j);
            hm.m[0] |= (unsigned long long)(v & 1u) << j;
            hm.m[1] |= (unsigned long long)((v >> 1) & 1u) << j;
        }
        HalfWalk hw;
        for (hw.start(hm); !hw.done(td.nsteps); hw.next(hm)) {
            KTile kt;
            step_ktile(p, td, hw.j, kt);
            const View& kv = p.view[kt.view];
            for (int rr = 0; rr < 128; ++rr) {
                const int rsub = rr / qv.R;
                const int ro = td.r0 + (rr - rsub * qv.R);
                const int rc = td.a0 + rsub;
                const bool row_valid = (rr < qv.R * qv.CH) && (rc <= td.a1) && (ro < qv.Z);
                int lo, hi;
                row_interval(kv, kt, rc, ro, rr, row_valid, lo, hi, kv.diag);
                if (!row_valid || hi <= lo) continue;
                for (int col = (lo > 64 * hw.h ? lo : 64 * hw.h); col < hi && col < 64 * hw.h + 64; ++col) {
                    const int ksub = col / kv.R;
                    const int64_t key = kt.r0 + (col - ksub * kv.R);
                    if (ksub == 0 && ro < l && key < W) {
                        uint8_t& c = counts[(int64_t)ro * W + key];
                        if (c < 255) ++c;
                    } else {
                        counts[0] = 255;   // a column outside the cache: never allowed
                    }
                }
            }
        }
    }
}

// The same count, taken from the key-tile side of the plan (the backward's dK/dV pass).
void plan_coverage_by_key_host(const Layout& L, uint8_t* counts) {
    FwdParams p{};
    make_plan(L, 1, 1, &p);
    memset(counts, 0, (size_t)L.S * L.S);
    for (int rank = 0; rank < p.total_tiles; ++rank) {
        KeyTileDesc kd;
        decode_key_tile(p, rank, kd);
        const View& kv = p.view[kd.view];
        HalfMasks hm{{0, 0}};
        for (int j = 0; j < kd.nsteps && j < 64; ++j) {
            const unsigned v = visited_qhalves(p, kd, j);
            hm.m[0] |= (unsigned long long)(v & 1u) << j;
            hm.m[1] |= (unsigned long long)((v >> 1) & 1u) << j;
        }
        HalfWalk hw;
        for (hw.start(hm); !hw.done(kd.nsteps); hw.next(hm)) {
            QTile qt;
            step_qtile(p, kd, hw.j, qt);
            const View& qv = p.view[qt.view];
            for (int kr = 0; kr < 128; ++kr) {
                const int ksub = kr / kv.R;
                const int ko = kd.r0 + (kr - ksub * kv.R);
                const int kc = kd.a0 + ksub;
                const bool key_valid = (kr < kv.R * kv.CH) && (kc <= kd.a1) && (ko < kv.Z);
                int lo, hi;
                col_interval(qv, qt, kc, ko, kr, key_valid, lo, hi);
                if (!key_valid || hi <= lo) continue;
                const int64_t gcol = (int64_t)kc * L.s + kv.zone_row0 + ko;
                for (int row = (lo > 64 * hw.h ? lo : 64 * hw.h); row < hi && row < 64 * hw.h + 64; ++row) {
                    const int rsub = row / qv.R;
                    const int ro = qt.r0 + (row - rsub * qv.R);
                    const int rc = qt.a0 + rsub;
                    const int64_t grow = (int64_t)rc * L.s + qv.zone_row0 + ro;
                    if (gcol < L.S && grow >= 0 && grow < L.S) {
                        uint8_t& c = counts[grow * L.S + gcol];
                        if (c < 255) ++c;
                    }
                }
            }
        }
    }
}

}  // namespace loma
