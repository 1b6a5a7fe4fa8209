// Host-side tree flattener (see ets_flatten.hpp).
#include "ets_flatten.hpp"

#include <algorithm>
#include <climits>
#include <cmath>
#include <functional>
#include <numeric>

namespace ets {

void tree_init(Tree& t, const FlattenParams& p, int64_t pages_per_layer) {
    t = Tree();
    t.free_heap.resize((size_t)pages_per_layer);
    for (int64_t i = 0; i < pages_per_layer; ++i) t.free_heap[(size_t)i] = (int32_t)(pages_per_layer - 1 - i);   // falling: the lowest id is at the back
    t.len.assign((size_t)p.num_layers, {});
    t.node_page_off.assign(1, 0);
    t.node_leaf_off.assign(1, 0);
    t.leaf_path_off.assign(1, 0);
    t.leaf_slot_off.assign(1, 0);
    t.worker_off.assign((size_t)std::max(1, p.n_workers) + 1, 0);
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

    // `t` may be an object that an earlier build filled: everything is set again below, and vectors that keep
    // their capacity save the allocations (and the page faults of fresh memory) of a rebuild.
    t.items.clear();
    t.n_narrow_items = 0;
    t.n_segments = t.n_chunks = t.n_partial_slots = 0;
    t.chunk_pages_used = 0;
    t.path_items = false;
    t.n_nodes = n_nodes;
    t.n_leaves = n_leaves;
    t.parent.assign(parent, parent + n_nodes);
    t.cap.assign(cap_tokens, cap_tokens + n_nodes);
    t.leaf_node.assign(leaf_node, leaf_node + n_leaves);
    const int32_t L = p.num_layers;
    t.len.resize((size_t)L);
    for (auto& v : t.len) v.assign((size_t)n_nodes, 0);

    // ---- pages: release what nobody keeps, then allocate in node order (lowest ids first)
    std::vector<int32_t> need((size_t)n_nodes);
    for (int32_t i = 0; i < n_nodes; ++i) need[i] = ceil_div(cap_tokens[i], p.page_size);
    if (keep_pages_of) {
        for (int32_t i = 0; i < n_nodes; ++i) {
            int32_t o = keep_pages_of[i];
            if (o < 0) continue;
            int32_t have = prev.node_page_off[o + 1] - prev.node_page_off[o];
            claimed_old[o] = std::min(have, need[i]);
        }
        for (int32_t l = 0; l < L; ++l) {
            int32_t* dst = t.len[l].data();
            const int32_t* src = prev.len[l].data();
            for (int32_t i = 0; i < n_nodes; ++i)
                if (keep_pages_of[i] >= 0) dst[i] = std::min(src[keep_pages_of[i]], cap_tokens[i]);
        }
    }
    // free pages, ids falling, so that the lowest is taken from the back; what this build releases is merged in
    {
        std::vector<int32_t> released;
        for (int32_t o = 0; o < n_prev; ++o) {
            int32_t keepn = std::max(claimed_old[o], 0);
            for (int32_t j = prev.node_page_off[o] + keepn; j < prev.node_page_off[o + 1]; ++j) released.push_back(prev.page_ids[j]);
        }
        if (released.empty()) {
            t.free_heap = prev.free_heap;
        } else {
            std::sort(released.begin(), released.end(), std::greater<int32_t>());
            t.free_heap.resize(prev.free_heap.size() + released.size());
            std::merge(prev.free_heap.begin(), prev.free_heap.end(), released.begin(), released.end(), t.free_heap.begin(),
                       std::greater<int32_t>());
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
            got = claimed_old[o];
            std::copy_n(prev.page_ids.data() + prev.node_page_off[o], got, t.page_ids.data() + w);
        }
        for (; got < need[i]; ++got) {
            if (t.free_heap.empty()) { err = "page pool exhausted at node " + std::to_string(i); return F_EXHAUSTED; }
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
    std::vector<int32_t> seg_last;                 // last node of each segment so far
    std::vector<int32_t> seg_next((size_t)n_nodes, -1);   // the segment's next node towards the leaves
    for (int32_t i = 0; i < n_nodes; ++i) {
        if (g[i] == 0) continue;
        int32_t pa = parent[i];
        if (pa >= 0 && g[pa] == g[i]) {
            seg_of[i] = seg_of[pa];
            seg_next[seg_last[seg_of[i]]] = i;
            seg_last[seg_of[i]] = i;
        } else {
            seg_of[i] = (int32_t)seg_head.size();
            seg_head.push_back(i);
            seg_last.push_back(i);
        }
    }
    const int32_t n_seg = (int32_t)seg_head.size();
    t.n_segments = n_seg;

    // ---- units (page slots) per segment
    std::vector<int32_t> seg_unit_off((size_t)n_seg + 1, 0);
    for (int32_t s = 0; s < n_seg; ++s) {
        int32_t cnt = 0;
        for (int32_t v = seg_head[s]; v >= 0; v = seg_next[v]) cnt += need[v];
        seg_unit_off[s + 1] = seg_unit_off[s] + cnt;
    }
    const int64_t n_units = seg_unit_off[n_seg];
    t.unit.resize((size_t)n_units * 4);
    for (int32_t s = 0; s < n_seg; ++s) {
        int32_t* u = t.unit.data() + 4 * (size_t)seg_unit_off[s];
        for (int32_t v = seg_head[s]; v >= 0; v = seg_next[v]) {
            const int32_t* pg = t.page_ids.data() + t.node_page_off[v];
            for (int32_t j = 0, nv = need[v]; j < nv; ++j, u += 4) {
                u[0] = pg[j];
                u[1] = v;
                u[2] = j * p.page_size;
                u[3] = 0;
            }
        }
    }

    // ---- narrow work queue.  A run is the page slots of one segment for one (kv head, leaf tile).
    // Runs are cut into pieces of at most `cap` page slots (at most 32: one lane per slot); a piece is
    // one work item.  The resident warps of the attention kernel take item w first (w = warp index)
    // and then claim the following items one by one from a shared counter, so the queue is ordered
    // longest piece first and its last pieces are cut shorter: whichever warp is early takes more.
    // The pieces of one (segment part) for all heads and leaf tiles stay adjacent in the queue: they
    // are claimed at about the same time, so the re-read of K/V by the next leaf tile hits in L2.
    const int32_t leaves_per_tile = std::max(1, p.rows_per_item / std::max(1, p.gqa));
    const int32_t n_workers = std::max(1, p.n_workers);
    const int32_t max_run = std::min(32, p.chunk_pages > 0 ? p.chunk_pages : 32);
    // A very small tree is left to the narrow kernel alone: a second kernel and the latency of its items cost
    // more than the re-reads they save when a warp has only a handful of page slots to read anyway (measured on a
    // width-16 tree with chained launches: 24.7 us per step without, 27.8 us with the second kernel).
    bool wide_pays = p.wide_rows > 0;
    if (wide_pays && !p.path_items) {
        int64_t all_narrow = 0;   // (page slot, kv head, leaf tile) visits if every segment were narrow
        for (int32_t s = 0; s < n_seg; ++s)
            all_narrow += (int64_t)(seg_unit_off[s + 1] - seg_unit_off[s]) * p.num_kv_heads * ceil_div(g[seg_head[s]], leaves_per_tile);
        wide_pays = all_narrow > (int64_t)p.wide_min_work * n_workers;
    }
    // Which of the two kernels ends last decides where the limit should sit: a tree whose bytes are under
    // large query groups keeps the wide kernel busy after the narrow one has finished, and every group the
    // narrow kernel takes over shortens the call; a tree with little sharing has the narrow kernel on the
    // critical path and the wide kernel idle at the end.  Run times of both at the lower limit, from counts
    // (fits to device time stamps on a 148-SM GPU: a narrow warp needs 1.5 us per page-slot visit, a wide
    // item 7 us per 64-token stage including its share of prologue and epilogue, one item per SM at a time).
    int32_t wide_min_rows = p.wide_min_rows;
    if (wide_pays && !p.path_items && p.wide_alt_rows > wide_min_rows) {
        const int32_t wide_leaves = std::max(1, p.wide_rows / std::max(1, p.gqa));
        int64_t visits = 0, stages = 0;
        for (int32_t s = 0; s < n_seg; ++s) {
            const int32_t nu = seg_unit_off[s + 1] - seg_unit_off[s], gn = g[seg_head[s]], r = gn * p.gqa;
            if (r > p.rows_per_item && r >= wide_min_rows) stages += (int64_t)ceil_div(nu, 4) * p.num_kv_heads * ceil_div(gn, wide_leaves);
            else visits += (int64_t)nu * p.num_kv_heads * ceil_div(gn, leaves_per_tile);
        }
        const double t_narrow = 5.0 + 1.5 * (double)visits / n_workers;
        const double t_wide = 7.0 + 7.0 * (double)stages / std::max(1, n_workers / 8);
        if (t_wide > t_narrow) wide_min_rows = p.wide_alt_rows;
    }
    auto is_wide = [&](int32_t s) {
        const int32_t r = g[seg_head[s]] * p.gqa;
        return wide_pays && r > p.rows_per_item && r >= wide_min_rows;
    };
    struct Part { int32_t seg, begin, len; };
    // per narrow segment: page slots, pieces per part (heads x leaf tiles), mean weight of a page slot
    // over its leaf tiles, leaves
    struct SegInfo { int32_t seg, nu, mult, gn; double w; };
    std::vector<SegInfo> narrow;
    narrow.reserve((size_t)n_seg);
    for (int32_t s = 0; s < n_seg; ++s) {
        const int32_t nu = seg_unit_off[s + 1] - seg_unit_off[s];
        if (nu == 0 || is_wide(s) || p.path_items) continue;
        const int32_t gn = g[seg_head[s]];
        const int32_t tiles = ceil_div(gn, leaves_per_tile);
        double wsum = 0.0;
        for (int32_t l0 = 0; l0 < gn; l0 += leaves_per_tile)
            wsum += (std::min(leaves_per_tile, gn - l0) * p.gqa > 8 ? p.cost_rows16 : 1.0) * (l0 > 0 ? p.cost_reread : 1.0);
        narrow.push_back({s, nu, p.num_kv_heads * tiles, gn, wsum / tiles});
    }
    // The estimate below is evaluated for up to ten piece lengths; segments with the same number of page slots
    // behave alike in it, so they are summed up once (a tree has a thousand segments and a few dozen lengths).
    struct Bucket { int32_t nu; int64_t mult, gn; double w_mult, w_max, w_min; };
    std::vector<Bucket> buckets;
    {
        int32_t max_nu = 0;
        for (const SegInfo& q : narrow) max_nu = std::max(max_nu, q.nu);
        std::vector<int32_t> at((size_t)max_nu + 1, -1);
        for (const SegInfo& q : narrow) {
            if (at[q.nu] < 0) { at[q.nu] = (int32_t)buckets.size(); buckets.push_back({q.nu, 0, 0, 0.0, q.w, q.w}); }
            Bucket& k = buckets[at[q.nu]];
            k.mult += q.mult;
            k.gn += q.gn;
            k.w_mult += q.w * q.mult;
            k.w_max = std::max(k.w_max, q.w);
            k.w_min = std::min(k.w_min, q.w);
        }
    }
    // Estimated time of the queue for a piece length, in page-slot units: the mean load of a warp plus
    // half of a late piece, or the longest piece when that is more or when there are no more pieces than warps.
    auto estimate = [&](int32_t cap, int32_t tail_cap, int64_t& slots_needed) {
        double total = 0.0, longest = 0.0, shortest = 1e30;
        slots_needed = 0;
        int64_t pieces = 0;
        for (const Bucket& q : buckets) {
            const int32_t np_ = ceil_div(q.nu, cap);
            const double len = (double)q.nu / np_;
            total += (double)np_ * p.cost_item * q.mult + q.nu * q.w_mult;
            longest = std::max(longest, p.cost_item + std::ceil(len) * q.w_max);
            shortest = std::min(shortest, p.cost_item + std::min<double>(len, tail_cap) * q.w_min);
            pieces += (int64_t)np_ * q.mult;
            slots_needed += (int64_t)np_ * p.num_kv_heads * q.gn;
        }
        if (narrow.empty()) return 0.0;
        if (pieces <= n_workers) return longest;   // every piece has a warp of its own
        // the cut of the last pieces adds about one item per warp
        if (pieces > n_workers && tail_cap < cap) { total += p.cost_item * n_workers; slots_needed += (int64_t)n_workers * leaves_per_tile; }
        return std::max(total / n_workers + 0.5 * shortest, longest);
    };
    int32_t cap = 0, tail_cap = 0;
    {
        static const int32_t kCaps[] = {32, 24, 16, 12, 8, 6, 4, 3, 2, 1};
        double best = 0.0;
        int32_t prev_c = 0;
        int32_t longest_seg = 0;
        for (const SegInfo& q : narrow) longest_seg = std::max(longest_seg, q.nu);
        for (int32_t cand : kCaps) {
            const int32_t c = std::min(cand, max_run);
            if (c == prev_c) continue;
            // a piece length at or above the longest segment cuts nothing: the same queue as the previous candidate
            if (prev_c != 0 && c >= longest_seg && prev_c >= longest_seg) continue;
            prev_c = c;
            // Last pieces: a quarter of the piece length, at least 8 page slots; at least 12 when a warp gets fewer
            // than three pieces anyway (one width-64 tree: opening an item then costs more than the shorter tail
            // returns; measured 32.1 -> 30.9 and 39.7 -> 38.1 us per call on the two width-64 trees, while the
            // width-256 tree, 4.5 pieces per warp, loses 0.6 % with 12).
            int64_t pieces_c = 0;
            for (const Bucket& q : buckets) pieces_c += (int64_t)ceil_div(q.nu, c) * q.mult;
            const int32_t tc = p.tail_pages > 0 ? p.tail_pages : std::max(pieces_c < 3 * (int64_t)n_workers ? 12 : 8, c / 4);
            int64_t need_slots = 0;
            const double est = estimate(c, tc, need_slots);
            if (need_slots > p.max_partial_slots || need_slots > p.max_items) continue;
            if (cap == 0 || est < best * 0.98) { best = est; cap = c; tail_cap = tc; }
        }
        if (cap == 0) { err = "partial-result slots exceed the workspace bound"; return F_EXHAUSTED; }
        t.chunk_pages_used = cap;
    }
    std::vector<Part> best_parts;
    {
        // stable order by falling length (a piece holds at most 32 page slots): a counting sort
        std::vector<Part> sorted;
        auto sort_by_len = [&](std::vector<Part>& v) {
            size_t first[34] = {};
            for (const Part& q : v) ++first[32 - q.len + 1];
            for (int k = 1; k < 34; ++k) first[k] += first[k - 1];
            sorted.resize(v.size());
            for (const Part& q : v) sorted[first[32 - q.len]++] = q;
            v.swap(sorted);
        };
        auto cut = [](std::vector<Part>& out, int32_t seg, int32_t begin, int32_t len, int32_t c) {
            const int32_t np_ = (len + c - 1) / c;
            for (int32_t k = 0; k < np_; ++k) {
                const int32_t b = (int32_t)((int64_t)len * k / np_), e = (int32_t)((int64_t)len * (k + 1) / np_);
                out.push_back({seg, begin + b, e - b});
            }
        };
        std::vector<int32_t> mult_of((size_t)n_seg, 0);
        int64_t total_pieces = 0;
        for (const SegInfo& q : narrow) {
            mult_of[q.seg] = q.mult;
            cut(best_parts, q.seg, 0, q.nu, cap);
        }
        sort_by_len(best_parts);
        for (const Part& q : best_parts) total_pieces += mult_of[q.seg];
        if (tail_cap < cap && total_pieces > n_workers) {
            // the parts that hold the last n_workers pieces of the queue are cut down to tail_cap
            size_t first = best_parts.size();
            int64_t pieces = 0;
            while (first > 0 && pieces < n_workers) { --first; pieces += mult_of[best_parts[first].seg]; }
            std::vector<Part> tail;
            for (size_t k = first; k < best_parts.size(); ++k) cut(tail, best_parts[k].seg, best_parts[k].begin, best_parts[k].len, tail_cap);
            best_parts.resize(first);
            best_parts.insert(best_parts.end(), tail.begin(), tail.end());
            sort_by_len(best_parts);
        }
    }
    int64_t slots = 0;
    // Every run of items made below covers one query group (gn leaves, listed from leaf_list_begin) for all kv
    // heads: head h, leaf position i gets partial slot base + h * gn + i.  The runs are remembered and the
    // per-(leaf, kv head) slot lists are written from them at the end, once per leaf instead of once per item.
    struct GroupRun { int32_t leaf_list_begin, gn; int64_t base; };
    std::vector<GroupRun> runs;
    {
        size_t n_items_narrow = 0;
        for (const Part& q : best_parts) n_items_narrow += (size_t)p.num_kv_heads * ceil_div(g[seg_head[q.seg]], leaves_per_tile);
        t.items.reserve(n_items_narrow + 64);
    }
    runs.reserve(best_parts.size() + 64);
    for (const Part& q : best_parts) {
        const int32_t head_node = seg_head[q.seg];
        const int32_t gn = g[head_node];
        const int32_t tiles = ceil_div(gn, leaves_per_tile);
        runs.push_back({t.node_leaf_off[head_node], gn, slots});
        const size_t first = t.items.size();
        t.items.resize(first + (size_t)p.num_kv_heads * tiles);
        Item* it = t.items.data() + first;
        const int32_t unit_begin = seg_unit_off[q.seg] + q.begin, list = t.node_leaf_off[head_node];
        for (int32_t h = 0; h < p.num_kv_heads; ++h)
            for (int32_t l0 = 0; l0 < gn; l0 += leaves_per_tile, ++it) {
                it->unit_begin = unit_begin;
                it->unit_count = q.len;
                it->kv_head = h;
                it->leaf_list_begin = list + l0;
                it->n_leaves_tile = std::min(leaves_per_tile, gn - l0);
                it->slot_first = (int32_t)slots;
                it->segment = q.seg;
                it->reserved = (l0 + leaves_per_tile < gn) ? 1 : 0;   // bit 0: the next tile re-reads these pages
                slots += it->n_leaves_tile;
            }
    }
    if (slots > p.max_partial_slots) { err = "partial-result slots exceed the workspace bound"; return F_EXHAUSTED; }
    t.n_narrow_items = (int32_t)t.items.size();
    // static first assignment: warp w starts with item w
    t.worker_off.assign((size_t)n_workers + 1, 0);
    for (int32_t k = 0; k <= n_workers; ++k) t.worker_off[k] = std::min(k, t.n_narrow_items);

    // ---- wide items: segments whose query group exceeds one narrow tile go to the tcgen05 kernel,
    // one CTA per (piece of the segment, kv head, tile of up to wide_rows query rows)
    if (p.wide_rows > 0 && !p.path_items) {
        const int32_t wide_leaves = std::max(1, p.wide_rows / std::max(1, p.gqa));
        // Piece length: long pieces amortise a CTA's fixed cost (TMEM allocation, Q tile, epilogue) over
        // several stages, short ones spread a small amount of wide work over more SMs.  Start long and
        // halve while the wide kernel would launch fewer CTAs than there are SMs.
        const int32_t n_sm = std::max(1, n_workers / 8);
        auto wide_ctas = [&](int32_t piece_len) {
            int64_t n = 0;
            for (int32_t s = 0; s < n_seg; ++s) {
                const int32_t nu = seg_unit_off[s + 1] - seg_unit_off[s];
                if (nu == 0 || !is_wide(s)) continue;
                n += (int64_t)ceil_div(nu, piece_len) * p.num_kv_heads * ceil_div(g[seg_head[s]], wide_leaves);
            }
            return n;
        };
        int32_t piece = std::max(1, std::min(p.wide_max_units, p.chunk_pages > 0 ? p.chunk_pages : INT32_MAX));
        while (piece > 8 && wide_ctas(piece) < n_sm) piece = std::max(8, piece / 2);
        if (p.wide_piece > 0) piece = p.wide_piece;
        for (int32_t s = 0; s < n_seg; ++s) {
            const int32_t nu = seg_unit_off[s + 1] - seg_unit_off[s];
            if (nu == 0 || !is_wide(s)) continue;
            const int32_t head_node = seg_head[s];
            const int32_t gn = g[head_node];
            const int32_t n_pieces = ceil_div(nu, piece);
            for (int32_t pc = 0; pc < n_pieces; ++pc) {
                const int32_t ub = (int32_t)((int64_t)nu * pc / n_pieces), ue = (int32_t)((int64_t)nu * (pc + 1) / n_pieces);
                runs.push_back({t.node_leaf_off[head_node], gn, slots});
                for (int32_t h = 0; h < p.num_kv_heads; ++h)
                    for (int32_t l0 = 0; l0 < gn; l0 += wide_leaves) {
                        Item it;
                        it.unit_begin = seg_unit_off[s] + ub;
                        it.unit_count = ue - ub;
                        it.kv_head = h;
                        it.leaf_list_begin = t.node_leaf_off[head_node] + l0;
                        it.n_leaves_tile = std::min(wide_leaves, gn - l0);
                        it.slot_first = (int32_t)slots;
                        it.segment = s;
                        it.reserved = (l0 + wide_leaves < gn) ? 1 : 0;
                        t.items.push_back(it);
                        slots += it.n_leaves_tile;
                        if (slots > p.max_partial_slots) { err = "partial-result slots exceed the workspace bound"; return F_EXHAUSTED; }
                    }
            }
        }
    }
    // ---- path items (step prefill): one item per (node that leaves sit at, kv head, tile of its leaves) whose
    // page slots are the node's whole root-to-node path.  A dense tile then walks its path once with its
    // accumulator resident, gathers its queries once and leaves one partial per row; the ancestors' K/V is
    // read once per tile of every node below them, as with segment items, but mostly from L2.
    t.path_items = p.path_items;
    if (p.path_items) {
        t.items.clear();
        runs.clear();
        slots = 0;
        std::vector<int32_t> at_off((size_t)n_nodes + 1, 0);
        for (int32_t l = 0; l < n_leaves; ++l) ++at_off[leaf_node[l] + 1];
        for (int32_t v = 0; v < n_nodes; ++v) at_off[v + 1] += at_off[v];
        const int32_t ext = (int32_t)t.node_leaves.size();       // leaves grouped by their own node follow the groups
        t.node_leaves.resize((size_t)ext + n_leaves);
        {
            std::vector<int32_t> cur(at_off.begin(), at_off.end() - 1);
            for (int32_t l = 0; l < n_leaves; ++l) t.node_leaves[(size_t)ext + cur[leaf_node[l]]++] = l;
        }
        const int32_t wide_leaves = std::max(1, std::max(p.wide_rows, 128) / std::max(1, p.gqa));
        std::vector<int32_t> path;
        for (int pass = 0; pass < 2; ++pass) {                   // small groups first: they are the narrow items
            for (int32_t v = 0; v < n_nodes; ++v) {
                const int32_t nl = at_off[v + 1] - at_off[v];
                if (nl == 0) continue;
                const bool dense = nl * p.gqa > p.rows_per_item;
                if (dense != (pass == 1)) continue;
                path.clear();
                for (int32_t x = v; x >= 0; x = parent[x]) path.push_back(x);
                const int32_t ub = (int32_t)(t.unit.size() / 4);
                for (auto it = path.rbegin(); it != path.rend(); ++it)
                    for (int32_t j = 0; j < need[*it]; ++j) {
                        t.unit.push_back(t.page_ids[t.node_page_off[*it] + j]);
                        t.unit.push_back(*it);
                        t.unit.push_back(j * p.page_size);
                        t.unit.push_back(0);
                    }
                const int32_t uc = (int32_t)(t.unit.size() / 4) - ub;
                if (uc == 0) continue;
                const int32_t per_tile = dense ? wide_leaves : leaves_per_tile;
                runs.push_back({ext + at_off[v], nl, slots});
                for (int32_t h = 0; h < p.num_kv_heads; ++h)
                    for (int32_t l0 = 0; l0 < nl; l0 += per_tile) {
                        Item it;
                        it.unit_begin = ub;
                        it.unit_count = uc;
                        it.kv_head = h;
                        it.leaf_list_begin = ext + at_off[v] + l0;
                        it.n_leaves_tile = std::min(per_tile, nl - l0);
                        it.slot_first = (int32_t)slots;
                        it.segment = -1;
                        it.reserved = 0;
                        t.items.push_back(it);
                        slots += it.n_leaves_tile;
                    }
            }
            if (pass == 0) t.n_narrow_items = (int32_t)t.items.size();
        }
        if (slots > p.max_partial_slots) { err = "partial-result slots exceed the workspace bound"; return F_EXHAUSTED; }
        for (int32_t k = 0; k <= n_workers; ++k) t.worker_off[k] = std::min(k, t.n_narrow_items);
    }
    t.n_chunks = (int64_t)t.items.size();
    t.n_partial_slots = slots;
    if ((int64_t)t.items.size() > p.max_items) { err = "work items exceed the workspace bound"; return F_EXHAUSTED; }

    // ---- per (leaf, kv head): the partial slots to merge, in item order.  A leaf meets the same runs for every
    // kv head, so its count is taken once and the H lists of a leaf lie one behind the other.
    const int32_t H = p.num_kv_heads;
    std::vector<int32_t> per_leaf((size_t)n_leaves, 0);
    for (const GroupRun& r : runs) {
        const int32_t* lv = t.node_leaves.data() + r.leaf_list_begin;
        for (int32_t i = 0; i < r.gn; ++i) ++per_leaf[lv[i]];
    }
    t.leaf_slot_off.resize((size_t)n_leaves * H + 1);
    {
        int32_t off = 0;
        for (int32_t l = 0; l < n_leaves; ++l)
            for (int32_t h = 0; h < H; ++h) {
                t.leaf_slot_off[(size_t)l * H + h] = off;
                off += per_leaf[l];
            }
        t.leaf_slot_off[(size_t)n_leaves * H] = off;
        t.leaf_slots.resize((size_t)off);
    }
    {
        std::vector<int32_t> cur((size_t)n_leaves, 0);
        for (const GroupRun& r : runs) {
            const int32_t* lv = t.node_leaves.data() + r.leaf_list_begin;
            for (int32_t i = 0; i < r.gn; ++i) {
                const int32_t l = lv[i], k = cur[l]++, n = per_leaf[l];
                int32_t* dst = t.leaf_slots.data() + t.leaf_slot_off[(size_t)l * H] + k;
                for (int32_t h = 0; h < H; ++h) dst[(size_t)h * n] = (int32_t)(r.base + (int64_t)h * r.gn + i);
            }
        }
    }
    return F_OK;
}

}  // namespace ets
