// Host-only self-test of the skinny kernel's schedule (SkinnyPlan / skinny_rect): for a
// sweep of (column tiles, K blocks, CTAs) it checks that the rectangles cover every
// (tile, K block) unit exactly once, that every tile is touched by exactly `nbands` CTAs
// with distinct band indices (= distinct scratch slots), that no CTA is empty, and that
// the largest rectangle stays close to the even share.  Built and run by the CPU
// test-suite; needs no GPU.
#include <cstdio>
#include <set>
#include <utility>
#include <vector>

#include "kernel_skinny.cuh"
#include "kernel_umma2.cuh"

using namespace optiml;

static double g_worst = 1.0;

static int check(int64_t T, int64_t KB, int sms, int64_t max_slots) {
    const SkinnyPlan p = make_skinny_plan(T, KB, sms, max_slots);
    if (p.G != p.S * p.T + p.G1 + p.G2 || p.G < 1 || p.G > sms) return 1;
    if (p.nbands != p.S + (p.G1 > 0) + (p.G2 > 0) || p.nbands < 1) return 2;
    if (p.nbands > 1 && (int64_t)p.nbands * T > max_slots) return 3;
    std::vector<int> cover((size_t)(T * KB), 0);
    std::set<std::pair<int, int>> band_tile;
    int64_t max_area = 0;
    for (int c = 0; c < p.G; ++c) {
        const SkinnyRect r = skinny_rect(p, c);
        if (r.t0 < 0 || r.t1 > T || r.t0 >= r.t1 || r.kb0 < 0 || r.kb1 > KB || r.kb0 >= r.kb1) return 4;
        if (r.band < 0 || r.band >= p.nbands) return 5;
        for (int t = r.t0; t < r.t1; ++t) {
            if (!band_tile.insert({r.band, t}).second) return 6;
            for (int kb = r.kb0; kb < r.kb1; ++kb) cover[(size_t)t * KB + kb] += 1;
        }
        const int64_t area = (int64_t)(r.t1 - r.t0) * (r.kb1 - r.kb0);
        if (area > max_area) max_area = area;
    }
    for (int v : cover)
        if (v != 1) return 7;
    if ((int64_t)band_tile.size() != (int64_t)p.nbands * T) return 8;
    const int used = sms < T * KB ? sms : (int)(T * KB);
    const double even = (double)(T * KB) / used;
    const double ratio = (double)max_area / even;
    const bool roomy = max_slots >= 3 * T;       // the scratch does not limit the banding
    if (roomy && T * KB >= 8 * (int64_t)sms && ratio > g_worst) g_worst = ratio;
    // with at least 8 units per CTA the banding must stay within 45 % of the even share (the
    // worst cases are T just above the CTA count and very few K blocks; typical shapes are
    // within a few per cent)
    if (roomy && T * KB >= 8 * (int64_t)sms && ratio > 1.45) return 9;
    return 0;
}

// The persistent CTA-pair kernel's work split: whole tiles round-robin, the tiles of the last
// partial round cut into K slices, one slice per pair.  Every (tile, K block) must be covered
// exactly once and every cut tile by exactly `split` slices with distinct indices.
static int check_pair_plan(int64_t M, int64_t N, int64_t K, int sms, int split_max) {
    const UmmaPlan p = make_umma2_plan(M, N, K, sms, split_max);
    const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
    if (p.grid < 1 || p.grid > sms / 2 || p.split < 1 || p.split > split_max) return 1;
    if (p.split == 1 ? (p.rem_tiles != 0 || p.full_tiles != tiles) : (p.full_tiles + p.rem_tiles != tiles)) return 2;
    if ((int64_t)p.rem_tiles * p.split > sms / 2) return 3;      // one slice per pair
    std::vector<int> cover((size_t)(tiles * p.num_kb), 0);
    std::set<std::pair<int, int>> slices;
    int most_items = 0;
    for (int c = 0; c < p.grid; ++c) {
        UmmaWork w;
        int i = 0;
        for (; umma2_work_item(p, c, i, w); ++i) {
            if (w.tm < 0 || w.tm >= p.tiles_m || w.tn < 0 || w.tn >= p.tiles_n || w.kb0 < 0 || w.kb0 >= w.kb1 || w.kb1 > p.num_kb)
                return 4;
            if (w.rem_idx >= 0) {
                if (w.rem_idx >= p.rem_tiles || w.chunk < 0 || w.chunk >= p.split) return 5;
                if (!slices.insert({w.rem_idx, w.chunk}).second) return 6;
            } else if (w.kb0 != 0 || w.kb1 != p.num_kb) {
                return 7;
            }
            for (int kb = w.kb0; kb < w.kb1; ++kb) cover[((size_t)w.tn * p.tiles_m + w.tm) * p.num_kb + kb] += 1;
            if (i > 1 << 20) return 8;
        }
        if (i > most_items) most_items = i;
    }
    for (int v : cover)
        if (v != 1) return 9;
    if ((int64_t)slices.size() != (int64_t)p.rem_tiles * p.split) return 10;
    // at most one slice after a pair's whole tiles
    const int64_t whole_rounds = (p.full_tiles + p.grid - 1) / p.grid;
    if (most_items > whole_rounds + 1) return 11;
    return 0;
}

int main() {
    {
        int bad_pairs = 0, n_pairs = 0;
        const int64_t Ms[] = {1, 256, 257, 512, 1024, 2304, 4096, 8192}, Ns[] = {8, 256, 520, 4096, 8192, 14336, 28672};
        const int64_t Ks[] = {8, 64, 256, 1032, 4096, 16384};
        for (int64_t M : Ms)
            for (int64_t N : Ns)
                for (int64_t K : Ks)
                    for (int sms : {2, 16, 132, 148})
                        for (int split_max : {1, 2, 3, 8}) {
                            const int rc = check_pair_plan(M, N, K, sms, split_max);
                            ++n_pairs;
                            if (rc) {
                                std::printf("FAIL pair plan M=%lld N=%lld K=%lld sms=%d split_max=%d code=%d\n", (long long)M,
                                            (long long)N, (long long)K, sms, split_max, rc);
                                ++bad_pairs;
                            }
                        }
        // 512 x 14336 x 4096 on 74 pairs: 112 whole tiles in two rounds (38 tiles cannot be cut for 74 pairs);
        // 4096^3: 222 whole tiles, 34 tiles in 2 slices
        const UmmaPlan a = make_umma2_plan(512, 14336, 4096, 148, 8), b = make_umma2_plan(4096, 4096, 4096, 148, 8);
        std::printf("pair plan 512x14336x4096: full=%d rem=%d split=%d grid=%d; 4096^3: full=%d rem=%d split=%d grid=%d\n", a.full_tiles,
                    a.rem_tiles, a.split, a.grid, b.full_tiles, b.rem_tiles, b.split, b.grid);
        std::printf("%d pair plans checked, %d wrong\n", n_pairs, bad_pairs);
        if (bad_pairs) return 1;
    }
    const int64_t Ts[] = {1, 2, 3, 7, 37, 56, 64, 73, 74, 75, 111, 112, 147, 148, 149, 160, 200, 296, 300, 1000, 5000};
    const int64_t KBs[] = {1, 2, 3, 5, 16, 17, 63, 64, 65, 128, 257};
    const int smss[] = {1, 2, 7, 132, 148};
    const int64_t slot_caps[] = {1024, 296};
    int bad = 0, n = 0;
    for (int64_t T : Ts)
        for (int64_t KB : KBs)
            for (int sms : smss)
                for (int64_t cap : slot_caps) {
                    const int rc = check(T, KB, sms, cap);
                    ++n;
                    if (rc) {
                        std::printf("FAIL T=%lld KB=%lld sms=%d cap=%lld code=%d\n", (long long)T, (long long)KB, sms,
                                    (long long)cap, rc);
                        ++bad;
                    }
                }
    // with the run-time model (192-row units of 51 KiB: 0.9 us each) the 16 x 14336 x 4096
    // problem runs as 112 whole tiles, four times the K as two balanced bands
    const SkinnyPlan c3t = make_skinny_plan(112, 22, 148, 1024, 0.9);
    const SkinnyPlan c3l = make_skinny_plan(112, 86, 148, 1024, 0.9);
    std::printf("c3 timed plan: nbands=%d G=%d; 4x K: nbands=%d G=%d\n", c3t.nbands, c3t.G, c3l.nbands, c3l.G);
    if (c3t.nbands != 1 || c3t.G != 112 || c3l.nbands != 2 || c3l.G != 148) ++bad;
    const SkinnyPlan c3 = make_skinny_plan(112, 64, 148, 1024);
    std::printf("c3 plan: S=%d k_split=%d G1=%d k_mid=%d G2=%d nbands=%d G=%d\n", c3.S, c3.k_split, c3.G1, c3.k_mid,
                c3.G2, c3.nbands, c3.G);
    const SkinnyPlan c2 = make_skinny_plan(64, 128, 148, 1024);
    std::printf("c2 plan: S=%d k_split=%d G1=%d k_mid=%d G2=%d nbands=%d G=%d\n", c2.S, c2.k_split, c2.G1, c2.k_mid,
                c2.G2, c2.nbands, c2.G);
    std::printf("worst max-area / even-share ratio: %.3f\n", g_worst);
    std::printf("%d plans checked, %d failed\n", n, bad);
    return bad ? 1 : 0;
}
