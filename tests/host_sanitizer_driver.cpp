// host-only functions of the library under AddressSanitizer / UBSan: tables from a gate map, plan building,
// append-token, drop-evicted, suffix-prefill tables, on random inputs (valid and invalid)
#include <cstdio>
#include <cstdlib>
#include <random>
#include <vector>
#include "rksc_internal.h"
int main() {
    std::mt19937 rng(7);
    int ok_plans = 0, rejected = 0;
    for (int trial = 0; trial < 400; ++trial) {
        const int P = 1 + rng() % 5, per = 1 + rng() % 6, B = P * per;
        const int Hkv = 1 << (rng() % 4), G = 1 + rng() % 8, hd = (rng() % 2) ? 128 : 64;
        std::vector<int32_t> so(P + 1, 0), sp, sn(P), po(B + 1, 0), pp, pn(B, 0), xo(B + 1, 0), xp, xn(B), map(B);
        int page = 0;
        for (int p = 0; p < P; ++p) { int n = rng() % 900; sn[p] = n; for (int i = 0; i < (n + 15) / 16; ++i) sp.push_back(page++); so[p + 1] = (int)sp.size(); }
        for (int b = 0; b < B; ++b) {
            const bool priv = (rng() % 10) < 3;
            map[b] = priv ? -1 : b / per;
            { int n = sn[b / per]; pn[b] = n; for (int i = 0; i < (n + 15) / 16; ++i) pp.push_back(page++); }
            po[b + 1] = (int)pp.size();
            int n = rng() % 300; xn[b] = n; for (int i = 0; i < (n + 15) / 16; ++i) xp.push_back(page++); xo[b + 1] = (int)xp.size();
        }
        rksc_layout L{Hkv * G, Hkv, hd, 16, 0.f, page + 3};
        const bool corrupt = trial % 7 == 6;
        if (corrupt && !xp.empty()) xp[rng() % xp.size()] = (rng() % 2) ? -1 : page + 100;   // a page id out of range
        rksc_tables t;
        if (rksc_tables_from_gate(B, P, map.data(), so.data(), sp.data(), sn.data(), po.data(), pp.data(), pn.data(), xo.data(), xp.data(), xn.data(), &t)) { printf("tables failed\n"); return 1; }
        rksc::HostPlan hp;
        const int st = rksc::build_host_plan(L, t, 148, &hp);
        if (st == RKSC_OK) ++ok_plans; else ++rejected;
        if (corrupt && !xp.empty() && st == RKSC_OK) { printf("corrupt table accepted\n"); return 1; }
        if (st == RKSC_OK) {
            // one decode step, an eviction and the prefill tables on top
            std::vector<int32_t> np(B), pg(B), sl(B);
            for (int b = 0; b < B; ++b) np[b] = page + 1 + b;
            rksc_layout L2 = L; L2.num_pool_blocks = page + 2 + B;
            rksc_tables t2;
            if (rksc_tables_append_token(&t, np.data(), &t2, pg.data(), sl.data()) == RKSC_OK) {
                rksc::HostPlan hp2;
                if (rksc::build_host_plan(L2, t2, 148, &hp2) != RKSC_OK) { printf("plan after append failed\n"); return 1; }
                std::vector<uint8_t> ev(t2.seg_block_off[t2.num_segments], 0);
                for (auto& e : ev) e = (rng() % 5) == 0;
                rksc_tables t3;
                if (rksc_tables_drop_evicted(&t2, ev.data(), &t3) == RKSC_OK) {
                    rksc::HostPlan hp3;
                    rksc::build_host_plan(L2, t3, 148, &hp3);
                    rksc_tables_free(&t3);
                }
                rksc_tables t4;
                if (rksc_tables_for_suffix_prefill(&t2, 1 + rng() % 16, &t4) == RKSC_OK) {
                    rksc::HostPlan hp4;
                    rksc::build_host_plan(L2, t4, 148, &hp4);
                    rksc_tables_free(&t4);
                }
                rksc_tables_free(&t2);
            }
        }
        rksc_tables_free(&t);
    }
    printf("plans built %d, tables rejected %d\n", ok_plans, rejected);
    return 0;
}
