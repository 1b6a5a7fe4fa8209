// Host-side tree flattener (see ets_flatten.hpp).
#include "ets_flatten.hpp"

#include <algorithm>
#include <functional>
#include <numeric>

namespace ets {

void tree_init(Tree& t, const FlattenParams& p, int64_t pages_per_layer) {
    t = Tree();
    t.free_heap.resize((size_t)pages_per_layer);
    std::iota(t.free_heap.begin(), t.free_heap.end(), 0);  // ascending = a valid min-heap
    t.len.assign((size_t)p.num_layers, {});
    t.node_page_off.assign(1, 0);
    t.node_leaf_off.assign(1, 0);
    t.leaf_path_off.assign(1, 0);
    t.leaf_slot_off.assign(1, 0);
}

static inline int32_t ceil_div(int32_t a, int32_t b) { return (a + b - 1) / b; }

int32_t tree_build(const Tree& prev, const FlattenParams& p, int32_t n_nodes, const int32_t* parent,
                   const int32_t* cap_tokens, const int32_t* keep_pages_of, int32_t n_leaves,
                   const int32_t* leaf_node, Tree& t, std::string& err) {
    // ---- validation
    if (n_nodes < 0 || n_leaves < 0) { err = "negative count"; return F_INVALID; }
    if ((n_nodes > 0 && (!parent || !cap_tokens)) || (n_leaves > 0 && !leaf_node)) {
        err = "null array"; return F_INVALID;
    }
    if (n_nodes > p.max_nodes) { err = "n_nodes exceeds max_nodes"; return F_EXHAUSTED; }
    if (n_leaves > p.max_leaves) { err = "n_leaves exceeds max_leaves"; return F_EXHAUSTED; }
    for (int32_t i = 0; i < n_nodes; ++i) {
        if (parent[i] < -1 || parent[i] >= i) {
            err = "parent[" + std::to_string(i) + "] must lie in [-1, i)"; return F_BAD_TREE;
        }
        if (cap_tokens[i] < 0) { err = "cap_tokens[" + std::to_string(i) + "] < 0"; return F_BAD_TREE; }
    }
    for (int32_t l = 0; l < n_leaves; ++l) {
        if (leaf_node[l] < 0 || leaf_node[l] >= n_nodes) {
            err = "leaf_node[" + std::to_string(l) + "] out of range"; return F_BAD_TREE;
        }
    }
    const int32_t n_prev = prev.n_nodes;
    std::vector<int32_t> claimed_old((size_t)n_prev, -1);  // pages of an old node that survive
    if (keep_pages_of) {
        for (int32_t i = 0; i < n_nodes; ++i) {
            int32_t o = keep_pages_of[i];
            if (o == -1) continue;
            if (o < 0 || o >= n_prev || claimed_old[o] != -1) {
                err = "keep_pages_of[" + std::to_string(i) + "] invalid or named twice"; return F_BAD_TREE;
            }
            claimed_old[o] = 0;
        }
    }

    t = Tree();
    t.n_nodes = n_nodes;
    t.n_leaves = n_leaves;
    t.parent.assign(parent, parent + n_nodes);
    t.cap.assign(cap_tokens, cap_tokens + n_nodes);
    t.leaf_node.assign(leaf_node, leaf_node + n_leaves);
    const int32_t L = p.num_layers;
    t.len.assign((size_t)L, std::vector<int32_t>((size_t)n_nodes, 0));

    // ---- pages: release what nobody keeps, then allocate in node order (lowest ids first)
    std::vector<int32_t> need((size_t)n_nodes);
    for (int32_t i = 0; i < n_nodes; ++i) need[i] = ceil_div(cap_tokens[i], p.page_size);
    if (keep_pages_of) {
        for (int32_t i = 0; i < n_nodes; ++i) {
            int32_t o = keep_pages_of[i];
            if (o < 0) continue;
            int32_t have = prev.node_page_off[o + 1] - prev.node_page_off[o];
            claimed_old[o] = std::min(have, need[i]);
            for (int32_t l = 0; l < L; ++l) t.len[l][i] = std::min(prev.len[l][o], cap_tokens[i]);
        }
    }
    t.free_heap = prev.free_heap;
    auto heap_cmp = std::greater<int32_t>();
    for (int32_t o = 0; o < n_prev; ++o) {
        int32_t keepn = std::max(claimed_old[o], 0);
        for (int32_t j = prev.node_page_off[o] + keepn; j < prev.node_page_off[o + 1]; ++j) {
            t.free_heap.push_back(prev.page_ids[j]);
            std::push_heap(t.free_heap.begin(), t.free_heap.end(), heap_cmp);
        }
    }
    t.node_page_off.assign((size_t)n_nodes + 1, 0);
    for (int32_t i = 0; i < n_nodes; ++i) t.node_page_off[i + 1] = t.node_page_off[i] + need[i];
    t.page_ids.resize((size_t)t.node_page_off[n_nodes]);
    for (int32_t i = 0; i < n_nodes; ++i) {
        int32_t w = t.node_page_off[i];
        int32_t got = 0;
        if (keep_pages_of && keep_pages_of[i] >= 0) {
            int32_t o = keep_pages_of[i];
            for (; got < claimed_old[o]; ++got) t.page_ids[w + got] = prev.page_ids[prev.node_page_off[o] + got];
        }
        for (; got < need[i]; ++got) {
            if (t.free_heap.empty()) { err = "page pool exhausted at node " + std::to_string(i); return F_EXHAUSTED; }
            std::pop_heap(t.free_heap.begin(), t.free_heap.end(), heap_cmp);
            t.page_ids[w + got] = t.free_heap.back();
            t.free_heap.pop_back();
        }
    }

    // ---- depth, groups, paths
    t.depth.assign((size_t)n_nodes, 0);
    for (int32_t i = 0; i < n_nodes; ++i) t.depth[i] = parent[i] < 0 ? 0 : t.depth[parent[i]] + 1;
    std::vector<int32_t> g((size_t)n_nodes, 0);
    int64_t n_path = 0;
    for (int32_t l = 0; l < n_leaves; ++l)
        for (int32_t v = leaf_node[l]; v >= 0; v = parent[v]) { ++g[v]; ++n_path; }
    if (n_path > p.max_path_entries) { err = "sum of path lengths exceeds max_path_entries"; return F_EXHAUSTED; }
    t.node_leaf_off.assign((size_t)n_nodes + 1, 0);
    for (int32_t i = 0; i < n_nodes; ++i) t.node_leaf_off[i + 1] = t.node_leaf_off[i] + g[i];
    t.node_leaves.resize((size_t)n_path);
    t.leaf_path_off.assign((size_t)n_leaves + 1, 0);
    t.leaf_path.resize((size_t)n_path);
    t.leaf_path_pos.resize((size_t)n_path);
    std::vector<int32_t> cursor((size_t)n_nodes, 0);
    for (int32_t l = 0; l < n_leaves; ++l) {
        int32_t d = t.depth[leaf_node[l]] + 1;
        int32_t base = t.leaf_path_off[l];
        t.leaf_path_off[l + 1] = base + d;
        int32_t k = d;
        for (int32_t v = leaf_node[l]; v >= 0; v = parent[v]) {
            --k;
            t.leaf_path[base + k] = v;
            t.leaf_path_pos[base + k] = cursor[v];
            t.node_leaves[t.node_leaf_off[v] + cursor[v]] = l;  // leaves ascend, so lists ascend
            ++cursor[v];
        }
    }

    // ---- segments: a node continues its parent's segment iff both have the same leaves below
    std::vector<int32_t> seg_of((size_t)n_nodes, -1);
    std::vector<int32_t> seg_head;                 // first node of each segment
    std::vector<std::vector<int32_t>> seg_nodes;   // nodes in root-to-leaf order
    for (int32_t i = 0; i < n_nodes; ++i) {
        if (g[i] == 0) continue;
        int32_t pa = parent[i];
        if (pa >= 0 && g[pa] == g[i]) {
            seg_of[i] = seg_of[pa];
            seg_nodes[seg_of[i]].push_back(i);
        } else {
            seg_of[i] = (int32_t)seg_head.size();
            seg_head.push_back(i);
            seg_nodes.push_back({i});
        }
    }
    const int32_t n_seg = (int32_t)seg_head.size();
    t.n_segments = n_seg;

    // ---- units (page slots) per segment
    std::vector<int32_t> seg_unit_off((size_t)n_seg + 1, 0);
    for (int32_t s = 0; s < n_seg; ++s) {
        int32_t cnt = 0;
        for (int32_t v : seg_nodes[s]) cnt += need[v];
        seg_unit_off[s + 1] = seg_unit_off[s] + cnt;
    }
    const int64_t n_units = seg_unit_off[n_seg];
    t.unit.resize((size_t)n_units * 4);
    for (int32_t s = 0; s < n_seg; ++s) {
        int32_t u = seg_unit_off[s];
        for (int32_t v : seg_nodes[s])
            for (int32_t j = 0; j < need[v]; ++j, ++u) {
                t.unit[4 * (size_t)u + 0] = t.page_ids[t.node_page_off[v] + j];
                t.unit[4 * (size_t)u + 1] = v;
                t.unit[4 * (size_t)u + 2] = j * p.page_size;
                t.unit[4 * (size_t)u + 3] = 0;
            }
    }

    // ---- chunking: enough (chunk, head) pairs to keep every worker busy several times over
    int32_t cp = p.chunk_pages;
    if (cp <= 0) {
        int64_t want_items = (int64_t)p.n_workers * 8;
        int64_t c = (n_units * p.num_kv_heads) / std::max<int64_t>(want_items, 1);
        cp = (int32_t)std::min<int64_t>(std::max<int64_t>(c, 8), 64);
    }
    t.chunk_pages_used = cp;
    const int32_t leaves_per_tile = std::max(1, p.rows_per_item / std::max(1, p.gqa));

    struct Chunk { int32_t ub, uc, seg, slot_base; };
    std::vector<Chunk> chunks;
    std::vector<int32_t> seg_chunk_off((size_t)n_seg + 1, 0);
    int64_t slots = 0;
    for (int32_t s = 0; s < n_seg; ++s) {
        int32_t nu = seg_unit_off[s + 1] - seg_unit_off[s];
        int32_t nc = std::max(1, ceil_div(nu, cp));   // a segment without pages still gets one (empty) chunk
        int32_t base = nu / nc, rem = nu % nc, ub = seg_unit_off[s];
        for (int32_t c = 0; c < nc; ++c) {
            int32_t uc = base + (c < rem ? 1 : 0);
            chunks.push_back({ub, uc, s, (int32_t)slots});
            slots += g[seg_head[s]];
            ub += uc;
        }
        seg_chunk_off[s + 1] = (int32_t)chunks.size();
    }
    if (slots > p.max_partial_slots) { err = "partial-result slots exceed the workspace bound"; return F_EXHAUSTED; }
    t.n_chunks = (int64_t)chunks.size();
    t.n_partial_slots = slots;

    // ---- items: (chunk, kv head, leaf tile); tiles of one (chunk, head) are adjacent so that
    // the re-reads of its K/V by later tiles hit in L2
    for (size_t c = 0; c < chunks.size(); ++c) {
        const Chunk& ch = chunks[c];
        int32_t head = seg_head[ch.seg];
        int32_t gn = g[head];
        for (int32_t h = 0; h < p.num_kv_heads; ++h)
            for (int32_t l0 = 0; l0 < gn; l0 += leaves_per_tile) {
                Item it;
                it.unit_begin = ch.ub;
                it.unit_count = ch.uc;
                it.kv_head = h;
                it.leaf_list_begin = t.node_leaf_off[head] + l0;
                it.n_leaves_tile = std::min(leaves_per_tile, gn - l0);
                it.slot_first = ch.slot_base + l0;
                it.chunk = (int32_t)c;
                it.reserved = 0;
                t.items.push_back(it);
            }
    }
    if ((int64_t)t.items.size() > p.max_items) { err = "work items exceed the workspace bound"; return F_EXHAUSTED; }

    // ---- per leaf: the partial slots to merge (one per chunk of every segment on its path)
    t.leaf_slot_off.assign((size_t)n_leaves + 1, 0);
    for (int32_t l = 0; l < n_leaves; ++l) {
        for (int32_t e = t.leaf_path_off[l]; e < t.leaf_path_off[l + 1]; ++e) {
            int32_t v = t.leaf_path[e];
            int32_t s = seg_of[v];
            if (seg_head[s] != v) continue;
            for (int32_t c = seg_chunk_off[s]; c < seg_chunk_off[s + 1]; ++c)
                t.leaf_slots.push_back(chunks[c].slot_base + t.leaf_path_pos[e]);
        }
        t.leaf_slot_off[l + 1] = (int32_t)t.leaf_slots.size();
    }
    return F_OK;
}

}  // namespace ets
