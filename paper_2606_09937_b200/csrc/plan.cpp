// Host-side integer work: tables from a gate map, table validation, sharing groups,
// KV chunking, workspace and block-mass layout.  No CUDA calls in this file.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>

#include "rksc_internal.h"

namespace rksc {

namespace {

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Relative cost of a work item for packing: streaming its pages plus a fixed start-up share.
inline int64_t item_cost(const WorkItem& it, int G) {
    const int nrt = ceil_div(it.num_sharers * G, 16);
    return (int64_t)it.num_pages * (8 + (nrt - 1)) + 64;
}

bool env_flag(const char* name) {
    const char* v = std::getenv(name);
    return v && v[0] && v[0] != '0';
}

bool csr_ok(const int32_t* off, int n) {
    if (off[0] != 0) return false;
    for (int i = 0; i < n; ++i)
        if (off[i + 1] < off[i]) return false;
    return true;
}

}  // namespace

int32_t build_host_plan(const rksc_layout& L, const rksc_tables& t, int num_sms, HostPlan* hp) {
    if (L.num_q_heads <= 0 || L.num_kv_heads <= 0 || L.num_pool_blocks <= 0) return RKSC_ERR_INVALID_ARG;
    if (L.num_q_heads % L.num_kv_heads != 0) return RKSC_ERR_INVALID_ARG;
    if (L.block_size != kBlock) return RKSC_ERR_UNSUPPORTED;
    if (L.head_dim != 64 && L.head_dim != 128) return RKSC_ERR_UNSUPPORTED;
    const int G = L.num_q_heads / L.num_kv_heads;
    if (G > kMaxRowsPerItem) return RKSC_ERR_UNSUPPORTED;   // one branch's heads of a KV head stay in one item
    if ((int64_t)L.num_pool_blocks * L.num_kv_heads * kBlock >= (int64_t)1 << 31) return RKSC_ERR_UNSUPPORTED;
    if (t.num_branches < 0 || t.num_segments < 0) return RKSC_ERR_INVALID_ARG;
    if (!t.seg_block_off || !t.br_seg_off) return RKSC_ERR_INVALID_ARG;
    const int B = t.num_branches, S = t.num_segments;
    if (S > 0 && !t.seg_num_tokens) return RKSC_ERR_INVALID_ARG;
    if (!csr_ok(t.seg_block_off, S) || !csr_ok(t.br_seg_off, B)) return RKSC_ERR_BAD_TABLE;
    const int total_pages = t.seg_block_off[S];
    const int total_refs = t.br_seg_off[B];
    if (total_pages > 0 && !t.seg_blocks) return RKSC_ERR_INVALID_ARG;
    if (total_refs > 0 && !t.br_segs) return RKSC_ERR_INVALID_ARG;

    for (int s = 0; s < S; ++s) {
        const int np = t.seg_block_off[s + 1] - t.seg_block_off[s];
        const int nt = t.seg_num_tokens[s];
        if (nt < 0 || np != ceil_div(nt, kBlock)) return RKSC_ERR_BAD_TABLE;
    }
    {
        // range checks without an early exit, so that the loops vectorise (26 k page ids on config 4)
        uint32_t bad = 0;
        const uint32_t nblk = (uint32_t)L.num_pool_blocks, ns = (uint32_t)S;
        for (int i = 0; i < total_pages; ++i) bad |= (uint32_t)((uint32_t)t.seg_blocks[i] >= nblk);
        for (int i = 0; i < total_refs; ++i) bad |= (uint32_t)((uint32_t)t.br_segs[i] >= ns);
        if (bad) return RKSC_ERR_BAD_TABLE;
    }

    HostPlan& P = *hp;
    P.reset();
    P.layout = L;
    P.B = B;
    P.S = S;
    P.G = G;
    P.seg_block_off.assign(t.seg_block_off, t.seg_block_off + S + 1);
    P.seg_blocks.assign(t.seg_blocks, t.seg_blocks + total_pages);
    P.seg_num_tokens.assign(t.seg_num_tokens, t.seg_num_tokens + S);

    // logical block counts and mass offsets
    P.br_nblk.assign(B, 0);
    P.mass_off.assign(B + 1, 0);
    for (int b = 0; b < B; ++b) {
        int64_t n = 0, tok = 0;
        for (int i = t.br_seg_off[b]; i < t.br_seg_off[b + 1]; ++i) {
            const int s = t.br_segs[i];
            n += P.seg_block_off[s + 1] - P.seg_block_off[s];
            tok += P.seg_num_tokens[s];
        }
        if (n >= ((int64_t)1 << 31)) return RKSC_ERR_UNSUPPORTED;
        P.br_nblk[b] = (int32_t)n;
        P.mass_off[b + 1] = P.mass_off[b] + n;
        P.duplicated_kv_tokens += tok;
    }
    P.mass_elems = P.mass_off[B] * L.num_q_heads;

    // sharing groups: for every segment the ascending list of (branch, mass position)
    P.seg_sharer_off.assign(S + 1, 0);
    for (int i = 0; i < total_refs; ++i) P.seg_sharer_off[t.br_segs[i] + 1]++;
    for (int s = 0; s < S; ++s) P.seg_sharer_off[s + 1] += P.seg_sharer_off[s];
    P.sharers.resize(total_refs);
    {
        std::vector<int32_t>& fill = P.scratch_a;
        fill.assign(P.seg_sharer_off.begin(), P.seg_sharer_off.end() - 1);
        for (int b = 0; b < B; ++b) {
            int64_t loff = 0;
            for (int i = t.br_seg_off[b]; i < t.br_seg_off[b + 1]; ++i) {
                const int s = t.br_segs[i];
                Sharer sh;
                sh.branch = b;
                sh.nblk = P.br_nblk[b];
                sh.mass_base = P.mass_off[b] * L.num_q_heads + loff;
                P.sharers[fill[s]++] = sh;
                loff += P.seg_block_off[s + 1] - P.seg_block_off[s];
            }
        }
    }

    // Work items.  A segment whose stacked rows (sharers x G) reach kTcMinRows goes to the
    // tensor-core (tcgen05) kernel in sharer blocks of up to 128 rows; the rest goes to the
    // warp-MMA kernel in blocks of up to 64 rows.  KV chunks are long enough that the partial
    // results stay a few percent of the KV bytes read (their size grows with the stacked rows)
    // and short enough that the persistent CTAs end together.
    const bool tc_ok = (L.head_dim == 128) && !env_flag("RKSC_DISABLE_TC");
    auto seg_rows_per_block = [&](int ns) {
        const bool tc = tc_ok && ns * G >= kTcMinRows;
        return std::max(1, (tc ? kTcMaxRows : kMaxRowsPerItem) / G);
    };
    int64_t total_units = 0;  // page-heads over all (segment, sharer block)
    for (int s = 0; s < S; ++s) {
        const int ns = P.seg_sharer_off[s + 1] - P.seg_sharer_off[s];
        const int np = P.seg_block_off[s + 1] - P.seg_block_off[s];
        if (ns == 0 || np == 0) continue;
        P.unique_kv_tokens += P.seg_num_tokens[s];
        total_units += (int64_t)np * L.num_kv_heads * ceil_div(ns, seg_rows_per_block(ns));
    }
    const int max_grid = std::max(1, num_sms) * kCtasPerSm;
    const int kMinChunk = 8;
    const int64_t fair = total_units / max_grid;                     // page-heads per CTA
    const int cap = (int)std::min<int64_t>(kMaxPagesPerItem, std::max<int64_t>(kMinChunk, fair * 2 / 3));
    const int base = (int)std::min<int64_t>(128, std::max<int64_t>(kMinChunk, fair / 6));

    // Items of the tensor-core kernel are as long as an SM's share of ALL the work (twice a CTA's share
    // at two warp-kernel CTAs per SM): that kernel pays for every item (epilogue, hand-over) and once
    // per CTA at its start, and the warp-MMA kernel, which starts at once on the SMs the tensor-core
    // kernel leaves free and on each of the others as the tensor-core CTA there ends, takes up the
    // slack of an uneven split.  Measured over long-context shapes (8 k - 64 k shared prefix, 8 - 32
    // branches) this length was the best of 1 x ... 3 x a CTA's share (8 % better than 1.5 x), and
    // neutral on the other configurations.
    const int tc_chunk = (int)std::min<int64_t>(kMaxPagesPerItem, std::max<int64_t>(kMinChunk, fair * 2));
    int64_t rows_total = 0;
    // Items are created in segment order and handed to the kernels sorted by (class, cost / 16), long
    // items first; the bucket of every item and the bucket counts are taken while the items are made,
    // so that the sort below is one scatter.  (A plan object is recycled with its vectors' capacity:
    // nothing is counted ahead.)
    constexpr int kBuckets = 1024;
    std::vector<int32_t>& bucket_of = P.scratch_a;
    bucket_of.clear();
    int32_t count[2][kBuckets + 1];
    std::memset(count, 0, sizeof(count));
    std::vector<WorkItem>& made = P.scratch_items;
    made.clear();
    for (int s = 0; s < S; ++s) {
        const int ns = P.seg_sharer_off[s + 1] - P.seg_sharer_off[s];
        const int np = P.seg_block_off[s + 1] - P.seg_block_off[s];
        if (ns == 0 || np == 0) continue;
        const int nsb = ceil_div(ns, seg_rows_per_block(ns));
        for (int sb = 0; sb < nsb; ++sb) {
            // balanced split of the sharers
            const int sh_lo = (int)((int64_t)ns * sb / nsb), sh_hi = (int)((int64_t)ns * (sb + 1) / nsb);
            const int rows = (sh_hi - sh_lo) * G;
            const int klass = (tc_ok && rows >= kTcMinRows) ? 1 : 0;
            int want = std::min(cap, std::max(base, 2 * rows));
            if (klass == 1) want = tc_chunk;
            const int nch = ceil_div(np, want);
            // chunk c covers pages [np * c / nch, np * (c + 1) / nch): one division per chunk, in 32 bits
            // where the product fits (64-bit divisions were a third of this loop's time)
            const bool narrow = (int64_t)np * nch < ((int64_t)1 << 31);
            auto cut = [&](int c) {
                return narrow ? (int)((uint32_t)np * (uint32_t)c / (uint32_t)nch) : (int)((int64_t)np * c / nch);
            };
            int p_hi = 0;
            for (int c = 0; c < nch; ++c) {
                const int p_lo = p_hi;
                p_hi = cut(c + 1);
                const int tok_lo = p_lo * kBlock;
                const int tok_hi = std::min(P.seg_num_tokens[s], p_hi * kBlock);
                WorkItem it{};
                it.seg = s;
                it.page_begin = P.seg_block_off[s] + p_lo;
                it.num_pages = p_hi - p_lo;
                it.num_tokens = tok_hi - tok_lo;
                it.sharer_begin = P.seg_sharer_off[s] + sh_lo;
                it.num_sharers = sh_hi - sh_lo;
                it.part_row_base = 0;  // set after sorting
                it.seg_page_begin = p_lo;
                it.klass = klass;
                const int64_t cost = item_cost(it, G);
                const int bkt = kBuckets - 1 - (int)std::min<int64_t>(kBuckets - 1, cost >> 4);   // small index = long item
                count[1 - klass][bkt + 1]++;
                it.kv_head = 0;   // one entry for the chunk's Hkv work items (see WorkItem)
                made.push_back(it);
                bucket_of.push_back(bkt);
                rows_total += (int64_t)rows * L.num_kv_heads;
            }
        }
    }
    if (rows_total >= ((int64_t)1 << 31)) return RKSC_ERR_UNSUPPORTED;

    // tensor-core items first, then warp-MMA items; within a class longest first, so that the
    // CTAs, which claim items in this order, finish together.  A counting sort on (class, cost / 16):
    // descending cost up to the bucket width is all the longest-first claiming needs, it keeps the
    // order of creation within a bucket, and it is linear in the number of items.
    {
        const size_t n = made.size();
        int32_t start[2][kBuckets];
        int32_t run = 0;
        for (int c = 0; c < 2; ++c)
            for (int b = 0; b < kBuckets; ++b) {
                start[c][b] = run;
                run += count[c][b + 1];
            }
        P.items.resize(n);
        for (size_t i = 0; i < n; ++i) P.items[start[1 - made[i].klass][bucket_of[i]]++] = made[i];
    }
    int32_t row = 0;
    P.num_tc_items = 0;
    const int Hkv = L.num_kv_heads;
    if ((int64_t)P.items.size() * Hkv >= ((int64_t)1 << 31)) return RKSC_ERR_UNSUPPORTED;
    for (auto& it : P.items) {
        it.part_row_base = row;
        row += it.num_sharers * G * Hkv;
        P.num_tc_items += it.klass * Hkv;
    }
    P.num_work_items = (int32_t)P.items.size() * Hkv;
    P.num_partial_rows = row;
    P.grid_tc = std::min(std::max(1, num_sms), P.num_tc_items);
    P.grid_warp = std::min(max_grid, P.num_work_items - P.num_tc_items);

    // merge lists: for every (branch, kv head) the partial rows (of head-in-group 0) to combine, in item
    // order.  A branch has the same number of parts under every KV head (an entry of the item array is
    // Hkv work items), so the parts are counted per branch and laid out head by head.
    const int nkeys = B * Hkv;
    {
        std::vector<int32_t>& cnt = P.scratch_b;   // parts per branch, then the next free position
        cnt.assign(B, 0);
        for (const auto& it : P.items)
            for (int i = 0; i < it.num_sharers; ++i) cnt[P.sharers[it.sharer_begin + i].branch]++;
        P.merge_off.resize(nkeys + 1);
        int32_t off = 0;
        for (int b = 0; b < B; ++b) {
            const int32_t n = cnt[b];
            for (int h = 0; h < Hkv; ++h) P.merge_off[b * Hkv + h] = off + h * n;
            off += n * Hkv;
            cnt[b] = 0;
        }
        P.merge_off[nkeys] = off;
        P.merge_rows.resize(off);
        for (const auto& it : P.items) {
            const int R = it.num_sharers * G;
            for (int i = 0; i < it.num_sharers; ++i) {
                const int b = P.sharers[it.sharer_begin + i].branch;
                const int pos = cnt[b]++;
                const int32_t n = P.merge_off[b * Hkv + 1] - P.merge_off[b * Hkv];   // the branch's parts per head
                for (int h = 0; h < Hkv; ++h)
                    P.merge_rows[P.merge_off[b * Hkv] + h * n + pos] = it.part_row_base + h * R + i * G;
            }
        }
    }

    // grid of the page-score kernel (RSBCM): 32 consecutive pages of one segment per CTA
    for (int s = 0; s < S; ++s) {
        const int n = P.seg_block_off[s + 1] - P.seg_block_off[s];
        for (int p0 = 0; p0 < n; p0 += 32) {
            P.score_chunks.push_back(s);
            P.score_chunks.push_back(p0);
        }
    }

    // workspace: partial outputs [rows][d] fp32, then partial log2-sum-exp [rows] fp32
    const size_t o_bytes = ((size_t)P.num_partial_rows * L.head_dim * sizeof(float) + 255) / 256 * 256;
    P.ws_lse_offset = o_bytes;
    P.workspace_bytes = o_bytes + ((size_t)P.num_partial_rows * sizeof(float) + 255) / 256 * 256;
    if (P.workspace_bytes == 0) P.workspace_bytes = 256;
    return RKSC_OK;
}

}  // namespace rksc

// ---------------------------------------------------------------------------------------------
// C ABI: tables from a gate map
// ---------------------------------------------------------------------------------------------

extern "C" RKSC_API int32_t rksc_tables_from_gate(int32_t B, int32_t P, const int32_t* map,
                                         const int32_t* shared_off, const int32_t* shared_pages, const int32_t* shared_ntok,
                                         const int32_t* priv_off, const int32_t* priv_pages, const int32_t* priv_ntok,
                                         const int32_t* sfx_off, const int32_t* sfx_pages, const int32_t* sfx_ntok,
                                         rksc_tables* out) {
    if (!out) return RKSC_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    if (B < 0 || P < 0) return RKSC_ERR_INVALID_ARG;
    if (B > 0 && (!map || !priv_off || !priv_ntok || !sfx_off || !sfx_ntok)) return RKSC_ERR_INVALID_ARG;
    if (P > 0 && (!shared_off || !shared_ntok)) return RKSC_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b)
        if (map[b] >= P) return RKSC_ERR_INVALID_ARG;

    std::vector<int32_t> shared_seg(P > 0 ? P : 1, -1);
    std::vector<int32_t> seg_off{0}, blocks, ntok, br_segs((size_t)2 * B);
    try {
        seg_off.reserve((size_t)P + 2 * (size_t)B + 1);
        ntok.reserve((size_t)P + 2 * (size_t)B);
        blocks.reserve((size_t)(P > 0 ? shared_off[P] : 0) + (size_t)(B > 0 ? priv_off[B] + sfx_off[B] : 0));
        auto add = [&](const int32_t* off, const int32_t* pages, const int32_t* nt, int i) {
            if (off[i + 1] > off[i]) blocks.insert(blocks.end(), pages + off[i], pages + off[i + 1]);
            seg_off.push_back((int32_t)blocks.size());
            ntok.push_back(nt[i]);
            return (int32_t)ntok.size() - 1;
        };
        std::vector<char> has(P > 0 ? P : 1, 0);
        for (int b = 0; b < B; ++b)
            if (map[b] >= 0) has[map[b]] = 1;
        for (int r = 0; r < P; ++r)
            if (has[r]) shared_seg[r] = add(shared_off, shared_pages, shared_ntok, r);
        for (int b = 0; b < B; ++b)
            if (map[b] < 0) br_segs[2 * b] = add(priv_off, priv_pages, priv_ntok, b);
            else br_segs[2 * b] = shared_seg[map[b]];
        for (int b = 0; b < B; ++b) br_segs[2 * b + 1] = add(sfx_off, sfx_pages, sfx_ntok, b);
    } catch (const std::bad_alloc&) {
        return RKSC_ERR_NOMEM;
    }
    const int S = (int)ntok.size();
    auto dup = [](const std::vector<int32_t>& v, size_t n) -> int32_t* {
        int32_t* p = (int32_t*)std::malloc(std::max<size_t>(1, n) * sizeof(int32_t));
        if (p && n) std::memcpy(p, v.data(), n * sizeof(int32_t));
        return p;
    };
    std::vector<int32_t> br_off(B + 1);
    for (int b = 0; b <= B; ++b) br_off[b] = 2 * b;
    int32_t* a0 = dup(seg_off, S + 1);
    int32_t* a1 = dup(blocks, blocks.size());
    int32_t* a2 = dup(ntok, S);
    int32_t* a3 = dup(br_off, B + 1);
    int32_t* a4 = dup(br_segs, (size_t)2 * B);
    if (!a0 || !a1 || !a2 || !a3 || !a4) {
        std::free(a0); std::free(a1); std::free(a2); std::free(a3); std::free(a4);
        return RKSC_ERR_NOMEM;
    }
    out->num_branches = B;
    out->num_segments = S;
    out->seg_block_off = a0;
    out->seg_blocks = a1;
    out->seg_num_tokens = a2;
    out->br_seg_off = a3;
    out->br_segs = a4;
    return RKSC_OK;
}

extern "C" RKSC_API void rksc_tables_free(rksc_tables* t) {
    if (!t) return;
    std::free((void*)t->seg_block_off);
    std::free((void*)t->seg_blocks);
    std::free((void*)t->seg_num_tokens);
    std::free((void*)t->br_seg_off);
    std::free((void*)t->br_segs);
    std::memset(t, 0, sizeof(*t));
}

// Tables after RSBCM eviction (Algorithm 4's effect on the block tables).
extern "C" RKSC_API int32_t rksc_tables_drop_evicted(const rksc_tables* in, const uint8_t* evicted, rksc_tables* out) {
    if (!in || !out) return RKSC_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    const int B = in->num_branches, S = in->num_segments;
    if (B < 0 || S < 0 || !in->seg_block_off || !in->br_seg_off) return RKSC_ERR_INVALID_ARG;
    if (S > 0 && !in->seg_num_tokens) return RKSC_ERR_INVALID_ARG;
    if (in->seg_block_off[0] != 0 || in->br_seg_off[0] != 0) return RKSC_ERR_BAD_TABLE;
    for (int s = 0; s < S; ++s) {
        const int64_t n = (int64_t)in->seg_block_off[s + 1] - in->seg_block_off[s];
        const int64_t nt = in->seg_num_tokens[s];
        if (n < 0 || nt < 0 || nt > n * rksc::kBlock || nt <= (n - 1) * rksc::kBlock) {
            if (!(n == 0 && nt == 0)) return RKSC_ERR_BAD_TABLE;
        }
    }
    for (int b = 0; b < B; ++b)
        if (in->br_seg_off[b + 1] < in->br_seg_off[b]) return RKSC_ERR_BAD_TABLE;
    const int64_t N = in->seg_block_off[S], R = in->br_seg_off[B];
    if (N > 0 && (!in->seg_blocks || !evicted)) return RKSC_ERR_INVALID_ARG;
    if (R > 0 && !in->br_segs) return RKSC_ERR_INVALID_ARG;
    auto alloc = [](size_t n) { return (int32_t*)std::malloc(std::max<size_t>(1, n) * sizeof(int32_t)); };
    int32_t* a0 = alloc((size_t)S + 1);
    int32_t* a1 = alloc((size_t)N);
    int32_t* a2 = alloc((size_t)S);
    int32_t* a3 = alloc((size_t)B + 1);
    int32_t* a4 = alloc((size_t)R);
    if (!a0 || !a1 || !a2 || !a3 || !a4) {
        std::free(a0); std::free(a1); std::free(a2); std::free(a3); std::free(a4);
        return RKSC_ERR_NOMEM;
    }
    int32_t kept = 0;
    a0[0] = 0;
    for (int s = 0; s < S; ++s) {
        const int lo = in->seg_block_off[s], hi = in->seg_block_off[s + 1];
        const int ntok = in->seg_num_tokens[s];
        int kept_tok = 0;
        for (int p = 0; p < hi - lo; ++p) {
            if (evicted[lo + p]) continue;
            a1[kept++] = in->seg_blocks[lo + p];
            kept_tok += std::min(rksc::kBlock, ntok - p * rksc::kBlock);
        }
        a0[s + 1] = kept;
        a2[s] = kept_tok;
    }
    std::memcpy(a3, in->br_seg_off, ((size_t)B + 1) * sizeof(int32_t));
    if (R > 0) std::memcpy(a4, in->br_segs, (size_t)R * sizeof(int32_t));
    out->num_branches = B;
    out->num_segments = S;
    out->seg_block_off = a0;
    out->seg_blocks = a1;
    out->seg_num_tokens = a2;
    out->br_seg_off = a3;
    out->br_segs = a4;
    return RKSC_OK;
}

// Tables that express the suffix prefill (Appendix "Stepwise Batched Decode", step 1) as a decode
// attention over B * s virtual branches; the numbering is fixed by the header.
extern "C" RKSC_API int32_t rksc_tables_for_suffix_prefill(const rksc_tables* in, int32_t s, rksc_tables* out) {
    if (!in || !out || s < 1) return RKSC_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    const int B = in->num_branches, S = in->num_segments;
    if (B < 0 || S < 0 || !in->seg_block_off || !in->br_seg_off) return RKSC_ERR_INVALID_ARG;
    if (S > 0 && !in->seg_num_tokens) return RKSC_ERR_INVALID_ARG;
    if ((int64_t)B * s >= ((int64_t)1 << 30) || (int64_t)S + (int64_t)B * (s + 1) >= ((int64_t)1 << 30))
        return RKSC_ERR_UNSUPPORTED;
    if (in->seg_block_off[0] != 0 || in->br_seg_off[0] != 0) return RKSC_ERR_BAD_TABLE;
    for (int sg = 0; sg < S; ++sg) {
        const int64_t n = (int64_t)in->seg_block_off[sg + 1] - in->seg_block_off[sg];
        const int64_t nt = in->seg_num_tokens[sg];
        if (n < 0 || nt < 0 || nt > n * rksc::kBlock || (n > 0 && nt <= (n - 1) * rksc::kBlock)) return RKSC_ERR_BAD_TABLE;
    }
    const int64_t N = in->seg_block_off[S], R = in->br_seg_off[B];
    if ((N > 0 && !in->seg_blocks) || (R > 0 && !in->br_segs)) return RKSC_ERR_INVALID_ARG;
    // sizes
    int64_t new_pages = N, new_refs = 0;
    for (int b = 0; b < B; ++b) {
        const int lo = in->br_seg_off[b], hi = in->br_seg_off[b + 1];
        if (hi < lo) return RKSC_ERR_BAD_TABLE;
        if (hi == lo) continue;
        for (int i = lo; i < hi; ++i)
            if (in->br_segs[i] < 0 || in->br_segs[i] >= S) return RKSC_ERR_BAD_TABLE;
        const int last = in->br_segs[hi - 1];
        const int64_t np = (int64_t)in->seg_block_off[last + 1] - in->seg_block_off[last];
        const int64_t T = in->seg_num_tokens[last];
        if (T < s) return RKSC_ERR_BAD_TABLE;
        const int64_t ncommon = (T - s) / rksc::kBlock;
        (void)np;
        for (int i = 0; i < s; ++i) new_pages += (T - s + i + 1 - ncommon * rksc::kBlock + rksc::kBlock - 1) / rksc::kBlock;
        new_pages += ncommon;
        new_refs += (int64_t)s * ((hi - lo) + 1);
    }
    if (new_pages >= ((int64_t)1 << 31) || new_refs >= ((int64_t)1 << 31)) return RKSC_ERR_UNSUPPORTED;
    const int S2 = S + B * (s + 1), B2 = B * s;
    auto alloc = [](size_t n) { return (int32_t*)std::malloc(std::max<size_t>(1, n) * sizeof(int32_t)); };
    int32_t* a0 = alloc((size_t)S2 + 1);
    int32_t* a1 = alloc((size_t)new_pages);
    int32_t* a2 = alloc((size_t)S2);
    int32_t* a3 = alloc((size_t)B2 + 1);
    int32_t* a4 = alloc((size_t)new_refs);
    if (!a0 || !a1 || !a2 || !a3 || !a4) {
        std::free(a0); std::free(a1); std::free(a2); std::free(a3); std::free(a4);
        return RKSC_ERR_NOMEM;
    }
    std::memcpy(a0, in->seg_block_off, ((size_t)S + 1) * sizeof(int32_t));
    if (N > 0) std::memcpy(a1, in->seg_blocks, (size_t)N * sizeof(int32_t));
    if (S > 0) std::memcpy(a2, in->seg_num_tokens, (size_t)S * sizeof(int32_t));
    int32_t pages = (int32_t)N, refs = 0;
    a3[0] = 0;
    for (int b = 0; b < B; ++b) {
        const int lo = in->br_seg_off[b], hi = in->br_seg_off[b + 1];
        const int seg0 = S + b * (s + 1);
        if (hi == lo) {
            for (int i = 0; i <= s; ++i) {
                a0[seg0 + i + 1] = pages;
                a2[seg0 + i] = 0;
            }
            for (int i = 0; i < s; ++i) a3[b * s + i + 1] = refs;
            continue;
        }
        const int last = in->br_segs[hi - 1];
        const int plo = in->seg_block_off[last], phi = in->seg_block_off[last + 1];
        const int T = in->seg_num_tokens[last];
        const int ncommon = (T - s) / rksc::kBlock;
        for (int p = 0; p < ncommon; ++p) a1[pages++] = in->seg_blocks[plo + p];
        a0[seg0 + 1] = pages;
        a2[seg0] = ncommon * rksc::kBlock;
        (void)phi;
        for (int i = 0; i < s; ++i) {
            const int nt = T - s + i + 1 - ncommon * rksc::kBlock;   // tokens of the tail part that token i sees
            const int npg = (nt + rksc::kBlock - 1) / rksc::kBlock;
            for (int p = 0; p < npg; ++p) a1[pages++] = in->seg_blocks[plo + ncommon + p];
            a0[seg0 + 1 + i + 1] = pages;
            a2[seg0 + 1 + i] = nt;
        }
        for (int i = 0; i < s; ++i) {
            for (int j = lo; j < hi - 1; ++j) a4[refs++] = in->br_segs[j];
            a4[refs++] = seg0;
            a4[refs++] = seg0 + 1 + i;
            a3[b * s + i + 1] = refs;
        }
    }
    out->num_branches = B2;
    out->num_segments = S2;
    out->seg_block_off = a0;
    out->seg_blocks = a1;
    out->seg_num_tokens = a2;
    out->br_seg_off = a3;
    out->br_segs = a4;
    return RKSC_OK;
}

// One decode step on the tables (Appendix "Stepwise Batched Decode", step 2): every branch with
// segments gains a token at the end of its last segment, which it must list alone.
extern "C" RKSC_API int32_t rksc_tables_append_token(const rksc_tables* in, const int32_t* new_pages, rksc_tables* out,
                                                     int32_t* page, int32_t* slot) {
    if (!in || !out) return RKSC_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    const int B = in->num_branches, S = in->num_segments;
    if (B < 0 || S < 0 || !in->seg_block_off || !in->br_seg_off) return RKSC_ERR_INVALID_ARG;
    if (B > 0 && (!page || !slot)) return RKSC_ERR_INVALID_ARG;
    if (S > 0 && !in->seg_num_tokens) return RKSC_ERR_INVALID_ARG;
    if (in->seg_block_off[0] != 0 || in->br_seg_off[0] != 0) return RKSC_ERR_BAD_TABLE;
    const int64_t N = in->seg_block_off[S], R = in->br_seg_off[B];
    if ((N > 0 && !in->seg_blocks) || (R > 0 && !in->br_segs)) return RKSC_ERR_INVALID_ARG;
    std::vector<int32_t> refs, grow;
    try {
        refs.assign((size_t)S, 0);
        grow.assign((size_t)S, -1);   // page appended to the segment, or -1
    } catch (const std::bad_alloc&) {
        return RKSC_ERR_NOMEM;
    }
    for (int64_t i = 0; i < R; ++i) {
        if (in->br_segs[i] < 0 || in->br_segs[i] >= S) return RKSC_ERR_BAD_TABLE;
        refs[in->br_segs[i]]++;
    }
    for (int s = 0; s < S; ++s) {
        const int64_t n = (int64_t)in->seg_block_off[s + 1] - in->seg_block_off[s];
        const int64_t nt = in->seg_num_tokens[s];
        if (n < 0 || nt < 0 || nt > n * rksc::kBlock || (n > 0 && nt <= (n - 1) * rksc::kBlock)) return RKSC_ERR_BAD_TABLE;
    }
    int64_t added = 0;
    for (int b = 0; b < B; ++b) {
        const int lo = in->br_seg_off[b], hi = in->br_seg_off[b + 1];
        if (hi < lo) return RKSC_ERR_BAD_TABLE;
        if (hi == lo) continue;
        const int s = in->br_segs[hi - 1];
        if (refs[s] != 1) return RKSC_ERR_BAD_TABLE;   // a shared segment cannot grow
        const int n = in->seg_block_off[s + 1] - in->seg_block_off[s];
        if (in->seg_num_tokens[s] == n * rksc::kBlock) {
            if (!new_pages || new_pages[b] < 0) return RKSC_ERR_INVALID_ARG;
            grow[s] = new_pages[b];
            ++added;
        }
    }
    if (N + added >= ((int64_t)1 << 31)) return RKSC_ERR_UNSUPPORTED;
    auto alloc = [](size_t n) { return (int32_t*)std::malloc(std::max<size_t>(1, n) * sizeof(int32_t)); };
    int32_t* a0 = alloc((size_t)S + 1);
    int32_t* a1 = alloc((size_t)(N + added));
    int32_t* a2 = alloc((size_t)S);
    int32_t* a3 = alloc((size_t)B + 1);
    int32_t* a4 = alloc((size_t)R);
    if (!a0 || !a1 || !a2 || !a3 || !a4) {
        std::free(a0); std::free(a1); std::free(a2); std::free(a3); std::free(a4);
        return RKSC_ERR_NOMEM;
    }
    int32_t w = 0;
    a0[0] = 0;
    for (int s = 0; s < S; ++s) {
        const int lo = in->seg_block_off[s], hi = in->seg_block_off[s + 1];
        if (hi > lo) std::memcpy(a1 + w, in->seg_blocks + lo, (size_t)(hi - lo) * sizeof(int32_t));
        w += hi - lo;
        if (grow[s] >= 0) a1[w++] = grow[s];
        a0[s + 1] = w;
        a2[s] = in->seg_num_tokens[s];
    }
    for (int b = 0; b < B; ++b) {
        const int lo = in->br_seg_off[b], hi = in->br_seg_off[b + 1];
        page[b] = slot[b] = -1;
        if (hi == lo) continue;
        const int s = in->br_segs[hi - 1];
        page[b] = a1[a0[s + 1] - 1];
        slot[b] = a2[s] % rksc::kBlock;
        a2[s] += 1;
    }
    std::memcpy(a3, in->br_seg_off, ((size_t)B + 1) * sizeof(int32_t));
    if (R > 0) std::memcpy(a4, in->br_segs, (size_t)R * sizeof(int32_t));
    out->num_branches = B;
    out->num_segments = S;
    out->seg_block_off = a0;
    out->seg_blocks = a1;
    out->seg_num_tokens = a2;
    out->br_seg_off = a3;
    out->br_segs = a4;
    return RKSC_OK;
}
