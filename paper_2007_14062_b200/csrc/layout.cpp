// Attention-graph layout of BigBird (arXiv 2007.14062, Sec. 2 and App. D) and the tile schedule the
// tensor-core kernel walks.  Host code only.
#include "layout.h"

#include <algorithm>
#include <atomic>
#include <new>

#include "../../include/bigbird.h"

namespace bigbird {
namespace {

// SplitMix64 (Steele, Lea, Flood 2014): the generator named by the layout spec in bigbird.h.
struct SplitMix64 {
    uint64_t s;
    explicit SplitMix64(uint64_t key) : s(key) {}
    uint64_t next() {
        s += 0x9E3779B97F4A7C15ull;
        uint64_t z = s;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        return z ^ (z >> 31);
    }
    // uniform integer in [0, m): floor(z * m / 2^64)
    uint64_t below(uint64_t m) { return (uint64_t)(((unsigned __int128)next() * m) >> 64); }
};

void global_flags(const bigbird_layout& L, std::vector<uint8_t>& is_global) {
    is_global.assign(L.nb, 0);
    if (L.mode == BIGBIRD_ETC) {
        for (int c = 0; c < L.g; ++c) is_global[c] = 1;             // Sec. 2, ETC: the g prepended tokens
    } else {
        const int first = (L.g + 1) / 2, last = L.g / 2;            // Sec. 2, ITC: a subset G of existing tokens
        for (int c = 0; c < first; ++c) is_global[c] = 1;
        for (int c = L.nb - last; c < L.nb; ++c) is_global[c] = 1;
    }
}

// Key blocks of one non-global query block: window (App. D item 2), global columns (item 3), random (item 1).
void sparse_row(const bigbird_layout& L, const std::vector<uint8_t>& is_global, int h, int j,
                std::vector<uint8_t>& mark, std::vector<int32_t>& cand, std::vector<int32_t>& out) {
    const int nb = L.nb, hw = (L.w - 1) / 2;
    std::fill(mark.begin(), mark.end(), 0);
    for (int c = std::max(0, j - hw); c <= std::min(nb - 1, j + hw); ++c) mark[c] = 1;
    for (int c = 0; c < nb; ++c)
        if (is_global[c]) mark[c] = 1;
    if (L.r > 0) {
        cand.clear();
        for (int c = 0; c < nb; ++c)
            if (!mark[c]) cand.push_back(c);
        const uint64_t m = cand.size();
        const uint64_t take = std::min<uint64_t>((uint64_t)L.r, m);
        SplitMix64 gen((L.seed << 40) ^ ((uint64_t)h << 20) ^ (uint64_t)j);
        for (uint64_t t = 0; t < take; ++t) {
            const uint64_t p = t + gen.below(m - t);
            std::swap(cand[t], cand[p]);
        }
        for (uint64_t t = 0; t < take; ++t) mark[cand[t]] = 1;
    }
    out.clear();
    for (int c = 0; c < nb; ++c)
        if (mark[c]) out.push_back(c);
}

}  // namespace

int build_layout_host(bigbird_layout* L, int chunk_steps) {
    const int nb = L->nb, H = L->H;
    std::vector<uint8_t> is_global, mark(nb);
    std::vector<int32_t> cand, row;
    global_flags(*L, is_global);

    // ---- CSR ------------------------------------------------------------------------------------
    L->row_ptr.assign(1, 0);
    L->col_idx.clear();
    for (int h = 0; h < H; ++h) {
        for (int j = 0; j < nb; ++j) {
            if (is_global[j]) {
                for (int c = 0; c < nb; ++c) L->col_idx.push_back(c);       // global rows attend everything
            } else {
                sparse_row(*L, is_global, h, j, mark, cand, row);
                L->col_idx.insert(L->col_idx.end(), row.begin(), row.end());
            }
            if (L->col_idx.size() > (size_t)INT32_MAX) return BIGBIRD_EUNSUPPORTED;
            L->row_ptr.push_back((int32_t)L->col_idx.size());
        }
    }

    // ---- the graph by key block (what the gradients of K and V walk) ----------------------------
    L->col_ptr.assign((size_t)H * nb + 1, 0);
    L->row_idx.assign(L->col_idx.size(), 0);
    for (int h = 0; h < H; ++h)
        for (int j = 0; j < nb; ++j)
            for (int32_t e = L->row_ptr[(size_t)h * nb + j]; e < L->row_ptr[(size_t)h * nb + j + 1]; ++e)
                ++L->col_ptr[(size_t)h * nb + L->col_idx[e] + 1];
    for (size_t i = 0; i < (size_t)H * nb; ++i) L->col_ptr[i + 1] += L->col_ptr[i];
    {
        std::vector<int32_t> fill(L->col_ptr.begin(), L->col_ptr.end() - 1);
        for (int h = 0; h < H; ++h)
            for (int j = 0; j < nb; ++j)                                     // ascending j: each list comes out sorted
                for (int32_t e = L->row_ptr[(size_t)h * nb + j]; e < L->row_ptr[(size_t)h * nb + j + 1]; ++e)
                    L->row_idx[fill[(size_t)h * nb + L->col_idx[e]]++] = j;
    }

    // ---- tile schedule ----------------------------------------------------------------------------
    // Query blocks are stacked two by two into 2b-row tiles: the global blocks among themselves (every key
    // block is attended by both halves), the others in ascending order.  A step is one key block together
    // with the halves of the tile that attend it.
    std::vector<int> gq, sq;
    for (int j = 0; j < nb; ++j) (is_global[j] ? gq : sq).push_back(j);
    const int n_gtiles = ((int)gq.size() + 1) / 2, n_stiles = ((int)sq.size() + 1) / 2;
    // default: a global tile of a long sequence is cut into parts of 32 key blocks, about the work of a few
    // sparse tiles, so that it does not outlast everything else; up to 96 blocks it stays whole
    if (chunk_steps <= 0) chunk_steps = nb <= 96 ? nb : 32;
    const int parts = (nb + chunk_steps - 1) / chunk_steps;
    L->max_parts = parts;
    L->split_tiles_per_head = parts > 1 ? n_gtiles : 0;
    L->heavy_items_per_head = n_gtiles * parts;
    L->items_per_head = L->heavy_items_per_head + n_stiles;
    L->items.clear();
    L->steps.clear();
    L->step_base.clear();
    L->split_tile_q.clear();
    for (int t = 0; t < n_gtiles && parts > 1; ++t) {
        L->split_tile_q.push_back(gq[2 * t]);
        L->split_tile_q.push_back(2 * t + 1 < (int)gq.size() ? gq[2 * t + 1] : kNoBlock);
    }
    std::vector<int32_t> la, lb, both, pa, pb;
    for (int h = 0; h < H; ++h) {
        const int32_t base = (int32_t)L->steps.size();
        L->step_base.push_back(base);
        auto rel = [&]() { return (int32_t)L->steps.size() - base; };
        for (int t = 0; t < n_gtiles; ++t) {
            const int32_t begin = rel();
            for (int c = 0; c < nb; ++c) L->steps.push_back(Step{c, kBothHalves});
            for (int p = 0; p < parts; ++p) {
                Item it{};
                it.qa = gq[2 * t];
                it.qb = 2 * t + 1 < (int)gq.size() ? gq[2 * t + 1] : kNoBlock;
                it.step_begin = begin + p * chunk_steps;
                it.step_count = std::min(chunk_steps, nb - p * chunk_steps);
                it.part = parts > 1 ? p : -1;
                it.nparts = parts;
                it.tile = t;
                L->items.push_back(it);
            }
        }
        for (int t = 0; t < n_stiles; ++t) {
            Item it{};
            it.qa = sq[2 * t];
            it.qb = 2 * t + 1 < (int)sq.size() ? sq[2 * t + 1] : kNoBlock;
            it.step_begin = rel();
            it.part = -1;
            it.nparts = 1;
            const int32_t* ra = &L->col_idx[L->row_ptr[(size_t)h * nb + it.qa]];
            const int na = L->row_ptr[(size_t)h * nb + it.qa + 1] - L->row_ptr[(size_t)h * nb + it.qa];
            la.assign(ra, ra + na);
            if (it.qb == kNoBlock) {
                for (int32_t c : la) L->steps.push_back(Step{c, kBothHalves});
            } else {
                const int32_t* rb = &L->col_idx[L->row_ptr[(size_t)h * nb + it.qb]];
                const int nbk = L->row_ptr[(size_t)h * nb + it.qb + 1] - L->row_ptr[(size_t)h * nb + it.qb];
                lb.assign(rb, rb + nbk);
                both.clear();
                pa.clear();
                pb.clear();
                size_t ia = 0, ib = 0;
                while (ia < la.size() || ib < lb.size()) {                   // merge of two ascending lists
                    if (ib == lb.size() || (ia < la.size() && la[ia] < lb[ib])) pa.push_back(la[ia++]);
                    else if (ia == la.size() || lb[ib] < la[ia]) pb.push_back(lb[ib++]);
                    else { both.push_back(la[ia]); ++ia; ++ib; }
                }
                // shared, upper-only and lower-only key blocks take turns, so that any run of three
                // consecutive steps gives both halves of the tile about the same amount of work
                const size_t ns = std::max(both.size(), std::max(pa.size(), pb.size()));
                for (size_t s = 0; s < ns; ++s) {
                    if (s < both.size()) L->steps.push_back(Step{both[s], kBothHalves});
                    if (s < pa.size()) L->steps.push_back(Step{pa[s], kUpperHalf});
                    if (s < pb.size()) L->steps.push_back(Step{pb[s], kLowerHalf});
                }
            }
            it.step_count = rel() - it.step_begin;
            L->items.push_back(it);
        }
    }
    L->items_abs = L->items;
    for (int h = 0; h < H; ++h)
        for (int i = 0; i < L->items_per_head; ++i) L->items_abs[(size_t)h * L->items_per_head + i].step_begin += L->step_base[h];
    return BIGBIRD_OK;
}

}  // namespace bigbird

extern "C" {

int bigbird_build_layout(int64_t N, int b, int w, int g, int r, uint64_t seed, int H, int mode,
                         bigbird_layout** out_layout) {
    if (!out_layout) return BIGBIRD_EINVAL;
    *out_layout = nullptr;
    if (N <= 0 || b <= 0 || N % b != 0) return BIGBIRD_EINVAL;
    const int64_t nb64 = N / b;
    if (nb64 >= (1 << 20) || H < 1 || H >= (1 << 20)) return BIGBIRD_EINVAL;     // stream-key field widths
    if (w < 1 || (w % 2) == 0 || g < 0 || g > nb64 || r < 0) return BIGBIRD_EINVAL;
    if (mode != BIGBIRD_ITC && mode != BIGBIRD_ETC) return BIGBIRD_EINVAL;
    if (seed >= (1ull << 24)) return BIGBIRD_EINVAL;                              // seed << 40 must not overflow
    bigbird_layout* L = new (std::nothrow) bigbird_layout();
    if (!L) return BIGBIRD_ENOMEM;
    L->N = N; L->b = b; L->w = w; L->g = g; L->r = r; L->H = H; L->mode = mode; L->seed = seed;
    L->nb = (int)nb64;
    static std::atomic<uint64_t> next_uid{1};
    L->uid = next_uid.fetch_add(1);
    int rc;
    try {
        rc = bigbird::build_layout_host(L, 0);
    } catch (const std::bad_alloc&) {
        rc = BIGBIRD_ENOMEM;
    }
    if (rc != BIGBIRD_OK) { delete L; return rc; }
    *out_layout = L;
    return BIGBIRD_OK;
}

int bigbird_layout_nnz(const bigbird_layout* L, int64_t* nnz) {
    if (!L || !nnz) return BIGBIRD_EINVAL;
    *nnz = (int64_t)L->col_idx.size();
    return BIGBIRD_OK;
}

int bigbird_layout_export(const bigbird_layout* L, int32_t* row_ptr, int32_t* col_idx) {
    if (!L || !row_ptr || !col_idx) return BIGBIRD_EINVAL;
    std::copy(L->row_ptr.begin(), L->row_ptr.end(), row_ptr);
    std::copy(L->col_idx.begin(), L->col_idx.end(), col_idx);
    return BIGBIRD_OK;
}

int bigbird_layout_export_transposed(const bigbird_layout* L, int32_t* col_ptr, int32_t* row_idx) {
    if (!L || !col_ptr || !row_idx) return BIGBIRD_EINVAL;
    std::copy(L->col_ptr.begin(), L->col_ptr.end(), col_ptr);
    std::copy(L->row_idx.begin(), L->row_idx.end(), row_idx);
    return BIGBIRD_OK;
}

const char* bigbird_strerror(int code) {
    switch (code) {
        case BIGBIRD_OK: return "ok";
        case BIGBIRD_EINVAL: return "invalid argument";
        case BIGBIRD_EUNSUPPORTED: return "unsupported shape or dtype";
        case BIGBIRD_ECUDA: return "CUDA call failed";
        case BIGBIRD_ETIMEOUT: return "bounded device wait expired";
        case BIGBIRD_ENOMEM: return "out of memory";
        case BIGBIRD_ELIMIT: return "problem exceeds the fixed scratch of the no-allocation entry point";
        case BIGBIRD_EINTERNAL: return "index check failed inside a kernel (checked build)";
        default: return "unknown error";
    }
}

}  // extern "C"

extern "C" int bigbird_layout_schedule(const bigbird_layout* L, int32_t* sizes, int32_t* items, int32_t* step_base,
                                       int32_t* steps) {
    if (!L || !sizes) return BIGBIRD_EINVAL;
    static_assert(sizeof(bigbird::Item) == 8 * sizeof(int32_t), "Item is exported as 8 int32");
    static_assert(sizeof(bigbird::Step) == 2 * sizeof(int32_t), "Step is exported as 2 int32");
    sizes[0] = L->items_per_head;
    sizes[1] = L->heavy_items_per_head;
    sizes[2] = (int32_t)L->steps.size();
    sizes[3] = L->H;
    if (items) std::copy((const int32_t*)L->items.data(), (const int32_t*)(L->items.data() + L->items.size()), items);
    if (step_base) std::copy(L->step_base.begin(), L->step_base.end(), step_base);
    if (steps) std::copy((const int32_t*)L->steps.data(), (const int32_t*)(L->steps.data() + L->steps.size()), steps);
    return BIGBIRD_OK;
}
