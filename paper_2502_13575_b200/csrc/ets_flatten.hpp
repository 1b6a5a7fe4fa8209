// Host-side tree flattener: page tables, query groups, leaf paths and the work
// decomposition for the attention kernels.  Pure C++ (no CUDA), so it can be exercised
// on a machine without a GPU.
//
// Semantics follow Section 4.1 and Appendix B of the paper: a node lies on a leaf's
// path iff the leaf descends from it, and all leaves through a node share its KV.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace ets {

struct FlattenParams {
    int32_t num_kv_heads = 1;
    int32_t gqa = 1;            // query heads per kv head
    int32_t page_size = 16;
    int32_t num_layers = 1;
    int32_t max_nodes = 0;
    int32_t max_leaves = 0;
    int64_t max_path_entries = 0;
    int64_t max_partial_slots = 0;
    int64_t max_items = 0;
    int32_t chunk_pages = 0;    // longest run of page slots in one item (0 = chosen by the builder; narrow items hold at most 32)
    int32_t tail_pages = 0;     // longest run in the last pieces of the narrow queue (0 = a quarter of the chosen length, at least 8)
    int32_t rows_per_item = 16; // query rows (leaves * gqa) one work item covers
    // cost model of the narrow kernel's queue, in units of one first-read page slot of a tile of
    // at most 8 query rows
    double cost_item = 2.0;      // opening an item (Q fragments, partial stores)
    double cost_rows16 = 1.2;    // factor for tiles of 9..16 query rows (two MMA column tiles); measured
    double cost_reread = 1.0;    // factor for second and later leaf tiles (their pages come from L2)
    int32_t wide_rows = 0;      // query rows one wide (tcgen05) item covers; 0 = no wide items
    int32_t wide_min_rows = 17; // smallest query group (in rows) that is treated as wide
    int32_t wide_min_work = 4;   // no wide items below this many page-slot visits per warp (counted as if all were narrow)
    int32_t wide_alt_rows = 0;   // if larger than wide_min_rows: the limit used instead when the wide kernel would end after the narrow one
    int32_t wide_max_units = 32; // longest page run of a wide item
    int32_t wide_piece = 0;      // page run of a wide item (0 = chosen by the builder)
    bool path_items = false;     // step prefill: items walk whole root-to-node paths (see tree_build)
    int32_t n_workers = 148 * 8; // warps the attention kernel keeps resident; they share the queue of narrow items
};

// One work item, as uploaded to the device (8 x int32).
struct Item {
    int32_t unit_begin, unit_count, kv_head, leaf_list_begin;
    int32_t n_leaves_tile, slot_first, segment, reserved;
};

struct Tree {
    int32_t n_nodes = 0, n_leaves = 0;
    std::vector<int32_t> parent, cap, leaf_node, depth;
    std::vector<int32_t> node_page_off, page_ids;
    std::vector<int32_t> node_leaf_off, node_leaves;
    std::vector<int32_t> leaf_path_off, leaf_path, leaf_path_pos;
    std::vector<std::vector<int32_t>> len;  // [layer][node]
    std::vector<int32_t> free_heap;         // free page ids in falling order: the lowest id is handed out first, from the back
    // work decomposition
    std::vector<int32_t> unit;              // 4 per unit: page, node, tok0, 0
    std::vector<Item> items;                // narrow items in queue order, then wide items
    int32_t n_narrow_items = 0;
    std::vector<int32_t> leaf_slot_off, leaf_slots;   // per (leaf, kv head)
    std::vector<int32_t> worker_off;                  // first item of warp w: [worker_off[w], worker_off[w+1]) (one or none)
    int64_t n_segments = 0, n_chunks = 0, n_partial_slots = 0;
    int32_t chunk_pages_used = 0;
    bool path_items = false;                // built for step prefill only
};

// Status codes mirror ets.h (kept numerically identical by a static_assert in the API file).
enum : int32_t { F_OK = 0, F_INVALID = -1, F_BAD_TREE = -2, F_EXHAUSTED = -3 };

// Fresh state: all pages free, no nodes.
void tree_init(Tree& t, const FlattenParams& p, int64_t pages_per_layer);

// Builds `next` from `prev` (which is left untouched; `next` must be another object).  `next` may hold an earlier
// build: all of it is overwritten and its vectors' capacity is reused.  On failure `next` is unspecified and
// `err` holds a message.
int32_t tree_build(const Tree& prev, const FlattenParams& p, int32_t n_nodes, const int32_t* parent,
                   const int32_t* cap_tokens, const int32_t* keep_pages_of, int32_t n_leaves,
                   const int32_t* leaf_node, Tree& next, std::string& err);

}  // namespace ets
