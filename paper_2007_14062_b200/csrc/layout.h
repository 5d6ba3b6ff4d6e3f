// Host-side attention-graph layout and the tile schedule derived from it.
#pragma once
#include <cstdint>
#include <mutex>
#include <vector>

namespace bigbird {

// One step of a tile's key sweep.  A tile stacks two query blocks (upper half = rows 0..b-1, lower half =
// rows b..2b-1).  A step names one key block and which halves of the tile attend it.
struct Step {
    int32_t c;      // key block
    int32_t who;    // kBothHalves, kUpperHalf or kLowerHalf
};
constexpr int32_t kBothHalves = 0;
constexpr int32_t kUpperHalf = 1;
constexpr int32_t kLowerHalf = 2;
constexpr int32_t kNoBlock = -1;

// One unit of work for a CTA: a tile of two query blocks and a contiguous range of steps.
struct Item {
    int32_t qa;          // query block of the upper half
    int32_t qb;          // query block of the lower half, or kNoBlock
    int32_t step_begin;  // index into the head's step array
    int32_t step_count;
    int32_t part;        // >= 0: this item is one chunk of a split tile and writes partial results to slot `part`
    int32_t nparts;      // number of chunks of the tile (1 = not split)
    int32_t tile;        // index of the split tile within the head (valid when nparts > 1)
    int32_t pad_;
};

struct DeviceLayout {
    int device = -1;
    int32_t* row_ptr = nullptr;
    int32_t* col_idx = nullptr;
    int32_t* col_ptr = nullptr;
    int32_t* row_idx = nullptr;
    Item* items = nullptr;
    Step* steps = nullptr;
    int32_t* split_tile_q = nullptr;   // [split_tiles_per_head * 2]
};

}  // namespace bigbird

struct bigbird_layout {
    int64_t N;
    int b, w, g, r, H, mode;
    uint64_t seed;
    uint64_t uid;                              // unique per handle for the life of the process, never 0
    int nb;
    // CSR over rows h*nb + j (the exported product)
    std::vector<int32_t> row_ptr;
    std::vector<int32_t> col_idx;
    // the same graph by key block: rows h*nb + c list, ascending, the query blocks that attend key block c
    std::vector<int32_t> col_ptr;
    std::vector<int32_t> row_idx;
    // tile schedule: per head the same number of items, heavy (global) items first
    int items_per_head = 0;
    int heavy_items_per_head = 0;   // leading items of each head that belong to global tiles
    int split_tiles_per_head = 0;   // global tiles cut into chunks (each needs a merge)
    int max_parts = 1;
    std::vector<bigbird::Item> items;          // [H * items_per_head], step_begin relative to the head's first step
    std::vector<bigbird::Item> items_abs;      // the same with step_begin made absolute (what the kernel reads)
    std::vector<int32_t> step_base;            // [H] offset of the head's steps in `steps`
    std::vector<bigbird::Step> steps;
    std::vector<int32_t> split_tile_q;         // [split_tiles_per_head * 2] query blocks (qa, qb) of each split tile
    // device copies, made on first use
    mutable std::mutex mu;
    mutable bigbird::DeviceLayout dev;
};

namespace bigbird {
// Builds CSR and schedule; returns 0 or a negative BIGBIRD_* code.  chunk_steps <= 0 picks the default.
int build_layout_host(bigbird_layout* L, int chunk_steps);
}
