// Host-side replay of the tensor-core kernel's tile plan.
#include <string.h>

#include "tile_plan.cuh"

namespace loma {

// counts[i*S + j] = number of (query tile, key tile) visits in which row i
// attends to column j.  A correct plan gives exactly the 0/1 mask of Eq. 2.
static HalfMasks host_half_masks(const FwdParams& p, const TileDesc& td) {
    HalfMasks hm{{0, 0}};
    for (int j = 0; j < td.nsteps && j < 64; ++j) {
        const unsigned v = visited_halves(p, td, j);
        hm.m[0] |= (unsigned long long)(v & 1u) << j;
        hm.m[1] |= (unsigned long long)((v >> 1) & 1u) << j;
    }
    return hm;
}

void plan_coverage_host(const Layout& L, uint8_t* counts) {
    FwdParams p{};
    make_plan(L, 1, 1, &p);
    memset(counts, 0, (size_t)L.S * L.S);
    // the kernel's unit of work is a pair of tiles; each tile of the pair walks its own steps
    for (int prank = 0; prank < p.total_pairs; ++prank) {
      PairDesc pd;
      decode_pair(p, prank, pd);
      for (int x = 0; x <= pd.nb; ++x) {
        const TileDesc& td = pd.td[x];
        const View& qv = p.view[td.view];
        // the same walk over visited halves as the kernel's roles take
        const HalfMasks hm = host_half_masks(p, td);
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
                row_interval(kv, kt, rc, ro, rr, row_valid, lo, hi);
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
}

// Replays, for every pair of the plan, the merged order of key-tile loads and the order in which the
// kernel issues its tensor-core instructions, and counts violations of what the kernel's roles rely on:
//   1. every tile's steps map to strictly increasing merged steps, every merged step has a source, and a
//      merged step that both tiles visit names the same key tile in both lists;
//   2. with a two-stage K/V ring that is filled in order (K0 V0 K1 V1 ...) and refilled after two releases,
//      the loader and the two tiles' issuers, each running as far as the ring lets it, all reach the end
//      (no wait can block for ever);
//   3. every K and V stage is released exactly twice, every tile issues one score product and one P.V
//      product per visited half, and the Q buffer is released once per tile.
int pair_plan_check_host(const Layout& L) {
    FwdParams p{};
    make_plan(L, 1, 1, &p);
    int bad = 0;
    for (int prank = 0; prank < p.total_pairs; ++prank) {
        PairDesc pd;
        decode_pair(p, prank, pd);
        const PairMap& pm = pd.pm;
        const int nm = pm.nmerged;
        if (nm <= 0) { ++bad; continue; }
        // 1. the merged order
        int visitors[2] = {0, 0};
        for (int x = 0; x <= pd.nb; ++x) {
            int prev = -1;
            for (int j = 0; j < pd.td[x].nsteps; ++j) {
                const int m = merged_index(pm, x, j);
                if (m <= prev || m >= nm || !visits_merged(pm, x, m)) ++bad;
                prev = m;
            }
        }
        for (int m = 0; m < nm; ++m) {
            int x, j;
            merged_source(pm, m, x, j);
            if (x < 0 || x > pd.nb || j < 0 || j >= pd.td[x].nsteps || merged_index(pm, x, j) != m) { ++bad; continue; }
            const bool va = visits_merged(pm, 0, m), vb = visits_merged(pm, 1, m);
            visitors[0] += va; visitors[1] += vb;
            if (!va && !vb) ++bad;
            if (va && vb) {
                if (!pd.nb) { ++bad; continue; }
                // find both tiles' steps with this merged index and compare their key tiles
                KTile ka, kb;
                int ja = -1, jb = -1;
                for (int jj = 0; jj < pd.td[0].nsteps; ++jj) if (merged_index(pm, 0, jj) == m) ja = jj;
                for (int jj = 0; jj < pd.td[1].nsteps; ++jj) if (merged_index(pm, 1, jj) == m) jb = jj;
                if (ja < 0 || jb < 0) { ++bad; continue; }
                step_ktile(p, pd.td[0], ja, ka);
                step_ktile(p, pd.td[1], jb, kb);
                if (ka.view != kb.view || ka.c0 != kb.c0 || ka.r0 != kb.r0) ++bad;
            }
        }
        if (visitors[0] != pd.td[0].nsteps || visitors[1] != (pd.nb ? pd.td[1].nsteps : 0)) ++bad;
        // 2, 3. the two tiles' instruction walks and the loads against the ring: three agents (the loader and
        // one issuer per tile), each blocked only by the ring; run them until nothing moves
        const HalfMasks hma = host_half_masks(p, pd.td[0]);
        const HalfMasks hmb = pd.nb ? host_half_masks(p, pd.td[1]) : hma;
        TileIssue ti[2];
        ti[0].start(pm, 0, hma, pd.td[0].nsteps);
        ti[1].start(pm, 1, hmb, pd.nb ? pd.td[1].nsteps : 0);
        int* rel_k = new int[nm]();
        int* rel_v = new int[nm]();
        int kl = 0, vl = 0;   // K / V tiles loaded so far, in the order K0 V0 K1 V1 ...
        int n_s[2] = {0, 0}, n_pv[2] = {0, 0}, n_q[2] = {0, 0};
        IssueAct pending[2];
        bool have[2] = {false, false};
        int last_m[2][2] = {{-1, -1}, {-1, -1}};   // per tile: last merged step of a P.V / of a score product
        for (long guard = 0;; ++guard) {
            if (guard > 16l * nm + 64) { ++bad; break; }
            bool moved = false;
            for (;;) {   // the loader
                // (the loader gives the second release itself where only one tile visits the step)
                if (kl == vl) {
                    if (kl >= nm || !(kl < 2 || rel_k[kl - 2] == 2)) break;
                    rel_k[kl] += 2 - (int)visits_merged(pm, 0, kl) - (int)visits_merged(pm, 1, kl);
                    ++kl;
                } else {
                    if (!(vl < 2 || rel_v[vl - 2] == 2)) break;
                    rel_v[vl] += 2 - (int)visits_merged(pm, 0, vl) - (int)visits_merged(pm, 1, vl);
                    ++vl;
                }
                moved = true;
            }
            for (int x = 0; x <= pd.nb; ++x) {
                for (;;) {
                    if (!have[x]) {
                        if (ti[x].done()) break;
                        ti[x].next(pending[x]);
                        have[x] = true;
                        int& lm = last_m[x][pending[x].is_s ? 1 : 0];
                        if (pending[x].m < lm || pending[x].m < 0 || pending[x].m >= nm) ++bad;
                        lm = pending[x].m;
                    }
                    const IssueAct& act = pending[x];
                    if (act.m < 0 || act.m >= nm) { have[x] = false; continue; }
                    if (act.is_s) {
                        if (kl <= act.m) break;   // waits for the K tile
                        ++n_s[x];
                        rel_k[act.m] += act.last_of_step;
                        if (act.last_s) ++n_q[x];
                    } else {
                        if (vl <= act.m) break;   // waits for the V tile (the probabilities always come)
                        ++n_pv[x];
                        rel_v[act.m] += act.last_of_step;
                    }
                    have[x] = false;
                    moved = true;
                }
            }
            if (!moved) break;
        }
        if (kl != nm || vl != nm || have[0] || have[1] || !ti[0].done() || (pd.nb && !ti[1].done())) ++bad;   // somebody is stuck
        for (int m = 0; m < nm; ++m) if (rel_k[m] != 2 || rel_v[m] != 2) ++bad;
        for (int x = 0; x <= pd.nb; ++x) {
            int events = 0;
            const HalfMasks& hm = x ? hmb : hma;
            HalfWalk hw;
            for (hw.start(hm); !hw.done(pd.td[x].nsteps); hw.next(hm)) ++events;
            if (n_s[x] != events || n_pv[x] != events || n_q[x] != 1) ++bad;
        }
        delete[] rel_k;
        delete[] rel_v;
    }
    return bad;
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
