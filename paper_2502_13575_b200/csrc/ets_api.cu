// C ABI of the library (see include/ets.h): context, workspace carving, table upload,
// launches.  No torch types, no exceptions across the boundary.
#include "../../include/ets.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstddef>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "ets_device.cuh"
#include "ets_flatten.hpp"

static_assert(ETS_ERR_INVALID_ARG == ets::F_INVALID && ETS_ERR_BAD_TREE == ets::F_BAD_TREE &&
                  ETS_ERR_POOL_EXHAUSTED == ets::F_EXHAUSTED, "status codes out of sync");
static_assert(sizeof(ets::Item) == 32 && sizeof(ets::DevItem) == 32, "item layout");

namespace {

constexpr int kStages = 3;        // pinned staging buffers for table uploads
constexpr int kDescSlots = 8;     // pinned/device descriptor slots for appends
constexpr int kTimingCap = 8192;  // decode calls that can be timed between two reads
constexpr int kMaxWorkers = 2048; // warp-workers of the attention kernel the tables are sized for
constexpr int kGroupLayers = 4;   // layers whose host buffers travel in one copy (ets_decode_step_host_layers)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {  // byte offsets inside the workspace
    size_t blob, blob_cap;
    size_t desc, desc_slot_bytes;
    size_t part_ml, part_o;
    size_t q_stage, out_stage, lse_stage, k_stage, v_stage;   // two of each, *_stride bytes apart
    size_t q_stride, lse_stride, kv_stride;
    size_t pk_stage, pk_stride;   // two areas for k_new | v_new | q of one call, contiguous
    size_t grp_in, grp_in_stride, grp_out, grp_out_stride, grp_lse, grp_lse_stride;   // two areas each for a group of layers
    size_t status;
    size_t stamps;
    size_t total;
    int64_t max_partial_slots, max_items, max_units;
    int32_t max_append_tokens;
};

bool config_ok(const ets_config* c, std::string& why) {
    if (!c) { why = "null config"; return false; }
    if (c->num_q_heads <= 0 || c->num_kv_heads <= 0 || c->num_q_heads % c->num_kv_heads) {
        why = "num_q_heads must be a positive multiple of num_kv_heads"; return false;
    }
    if (c->num_layers <= 0 || c->max_nodes <= 0 || c->max_leaves <= 0 || c->pages_per_layer <= 0 ||
        c->max_path_entries <= 0 || c->max_path_tokens <= 0 || c->max_append_tokens < 0) {
        why = "capacity bounds must be positive"; return false;
    }
    if (c->flags != 0) { why = "flags must be 0"; return false; }
    if (c->pages_per_layer > 0x7fffffffLL) { why = "pages_per_layer too large"; return false; }
    return true;
}

int32_t config_supported(const ets_config* c, std::string& why) {
    int g = c->num_q_heads / c->num_kv_heads;
    if (c->head_dim != 64 && c->head_dim != 128) { why = "head_dim must be 64 or 128"; return ETS_ERR_UNSUPPORTED; }
    if (c->page_size <= 0) { why = "page_size must be positive"; return ETS_ERR_UNSUPPORTED; }
    // the kernels are written for 16-token pages; a host-only context may flatten with any size
    if (c->device >= 0 && c->page_size != ets::kPageTokens) { why = "page_size must be 16"; return ETS_ERR_UNSUPPORTED; }
    if (!(g == 1 || g == 2 || g == 4 || g == 8 || g == 16)) {
        why = "num_q_heads/num_kv_heads must be 1, 2, 4, 8 or 16"; return ETS_ERR_UNSUPPORTED;
    }
    return ETS_OK;
}

Layout make_layout(const ets_config* c) {
    Layout L{};
    const int64_t path_pages = (int64_t)c->max_leaves * ((c->max_path_tokens + c->page_size - 1) / c->page_size) +
                               c->max_path_entries;
    // a partial slot belongs to one (item, leaf); items are (piece of a segment, kv head, leaf tile).  The
    // builder picks the piece length and falls back to longer pieces when a choice would not fit here.
    const int gqa = c->num_q_heads / c->num_kv_heads;
    L.max_partial_slots = (c->max_path_entries + (path_pages + 3) / 4) * c->num_kv_heads +
                          (int64_t)kMaxWorkers * 4 * (16 / gqa > 0 ? 16 / gqa : 1);
    L.max_items = L.max_partial_slots;
    L.max_units = c->pages_per_layer + path_pages;   // path items (step prefill) list a node's whole path
    L.max_append_tokens = c->max_append_tokens > 0 ? c->max_append_tokens : c->max_leaves;
    const size_t A = 1024;
    size_t blob = 0;
    blob += align_up((size_t)L.max_units * 16, 256);
    blob += align_up((size_t)L.max_items * 32, 256);
    blob += align_up(((size_t)c->max_nodes + 1) * 4, 256);          // node_page_off
    blob += align_up((size_t)c->pages_per_layer * 4, 256);          // page_ids
    blob += align_up(((size_t)c->max_path_entries + c->max_leaves) * 4, 256);   // node_leaves (+ leaves by own node)
    blob += align_up((size_t)c->max_leaves * 4, 256);               // leaf_node
    blob += align_up(((size_t)c->max_leaves * c->num_kv_heads + 1) * 4, 256);  // leaf_slot_off
    blob += align_up((size_t)L.max_partial_slots * 4, 256);         // leaf_slots
    blob += align_up((size_t)c->num_layers * c->max_nodes * 4, 256);  // node_len
    L.blob_cap = align_up(blob, A);
    size_t off = 0;
    L.blob = off; off += L.blob_cap;
    L.desc_slot_bytes = align_up((size_t)c->max_nodes * 16, 256);
    L.desc = off; off += align_up(L.desc_slot_bytes * (kDescSlots + 1), A);   // ring + the cached list
    const size_t rows = (size_t)L.max_partial_slots * gqa;
    L.part_ml = off; off += align_up(rows * 8, A);
    L.part_o = off; off += align_up(rows * c->head_dim * 4, A);
    const size_t qbytes = (size_t)c->max_leaves * c->num_q_heads * c->head_dim * 2;
    L.q_stride = align_up(qbytes, A);
    L.lse_stride = align_up((size_t)c->max_leaves * c->num_q_heads * 4, A);
    L.q_stage = off; off += 2 * L.q_stride;
    L.out_stage = off; off += 2 * L.q_stride;
    L.lse_stage = off; off += 2 * L.lse_stride;
    const size_t kvb = (size_t)L.max_append_tokens * c->num_kv_heads * c->head_dim * 2;
    L.kv_stride = align_up(kvb, A);
    L.k_stage = off; off += 2 * L.kv_stride;
    L.v_stage = off; off += 2 * L.kv_stride;
    L.pk_stride = align_up(2 * kvb + qbytes, A);
    L.pk_stage = off; off += 2 * L.pk_stride;
    L.grp_in_stride = align_up((size_t)kGroupLayers * (2 * kvb + qbytes), A);
    L.grp_in = off; off += 2 * L.grp_in_stride;
    L.grp_out_stride = align_up((size_t)kGroupLayers * qbytes, A);
    L.grp_out = off; off += 2 * L.grp_out_stride;
    L.grp_lse_stride = align_up((size_t)kGroupLayers * c->max_leaves * c->num_q_heads * 4, A);
    L.grp_lse = off; off += 2 * L.grp_lse_stride;
    L.status = off; off += A;
    L.stamps = off; off += align_up(sizeof(ets::Stamps), A);
    L.total = off;
    return L;
}

struct BlobOffsets {  // offsets of the packed tables of the current tree inside the device blob
    size_t units, items, node_page_off, page_ids, node_leaves, leaf_node, leaf_slot_off, leaf_slots, node_len, total;
    int32_t len_stride;
};

}  // namespace

struct ets_ctx {
    ets_config cfg{};
    ets::FlattenParams fp{};
    Layout lay{};
    ets::Tree tree;
    ets::Tree spare;   // the tree before the current one: the next build writes into it, reusing its memory
    ets::FlattenParams built{};   // the options the current tree was built with
    bool has_tree = false;
    bool host_only = true;
    int sm_count = 148;
    char* k_pool = nullptr;
    char* v_pool = nullptr;
    char* ws = nullptr;
    size_t layer_pool_bytes = 0;
    float scale_log2 = 0.f;
    BlobOffsets bo{};
    // pinned staging for table uploads
    char* stage_host[kStages] = {nullptr, nullptr, nullptr};
    cudaEvent_t stage_ev[kStages] = {nullptr, nullptr, nullptr};
    bool stage_used[kStages] = {false, false, false};
    int stage_next = 0;
    // pinned descriptor slots for appends
    int4* desc_host[kDescSlots] = {};
    cudaEvent_t desc_ev[kDescSlots] = {};
    bool desc_used[kDescSlots] = {};
    int desc_next = 0;
    // descriptors of the last short append (at most 8 tokens per node) stay on the device: a decode loop
    // repeats the same (node, count) list for every layer and step
    std::vector<int32_t> step_ones;   // n_new of ets_decode_step: one token per leaf
    std::vector<int32_t> cache_nodes, cache_nnew;
    bool cache_valid = false;
    cudaStream_t cache_stream = nullptr;
    cudaEvent_t cache_ev = nullptr;
    bool host_epoch_open = false;   // pipelined host calls: entry ordering already established
    int32_t* status_host = nullptr;  // pinned, target of the status read-back
    // host-buffer entry points: copies in, kernels and copies out run on three library streams so that
    // the transfers of one call overlap the kernels of its neighbours; staging areas alternate
    cudaStream_t st_in = nullptr, st_comp = nullptr, st_out = nullptr;
    cudaEvent_t ev_entry = nullptr, ev_q_in[2] = {}, ev_q_free[2] = {}, ev_comp[2] = {}, ev_out_free[2] = {};
    cudaEvent_t ev_kv_in[2] = {}, ev_kv_free[2] = {};
    bool q_used[2] = {false, false}, out_used[2] = {false, false}, kv_used[2] = {false, false};
    uint64_t n_host_decode = 0, n_host_append = 0, n_host_group = 0;
    cudaEvent_t ev_g_in[2] = {}, ev_g_free[2] = {}, ev_g_comp[2] = {}, ev_g_out[2] = {};
    bool g_used[2] = {false, false};
    bool opt_host_pipeline = false;   // host-buffer calls do not make the caller's stream wait; ets_host_join does
    bool host_pending = false;        // host-buffer work that the caller's stream has not been joined with yet
    cudaEvent_t ev_join_comp = nullptr, ev_join_out = nullptr;
    // second stream on which the wide-group kernel runs beside the narrow kernel when launches are not chained
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // options
    int32_t opt_chunk_pages = 0;
    int32_t opt_kernel = 0;
    bool opt_path_items = false;
    bool opt_overlap_append = false;
    bool opt_wide_set = false;   // the caller chose the wide threshold: no small-tree exception
    bool opt_packed_inputs = false;
    // One call's kernels are launched as a chain of programmatic dependents on one stream (see pdl_wait in
    // ets_device.cuh); 0: ordinary launches, the wide kernel on a second stream forked from the caller's.
    bool opt_chain = true;
    uint32_t opt_first_wait_polls = ets::kWaitPolls;
    // smallest query group (rows) sent to the wide kernel; 0 = never.  Measured on width-256 trees and on
    // eight width-64 trees: 33 is 1-2 % ahead of 49 and 65 per layer, 25 is 2-12 % and 17 15-20 % slower (below
    // ~32 rows the per-item latency of the wide kernel costs more than the re-reads by the narrow kernel that
    // it saves).
    int32_t opt_wide = 33;
    bool opt_timing = false;
    bool opt_stamps = false;          // device time stamps per kernel launch (ETS_OPT_TIMING = 2)
    // timing
    std::vector<cudaEvent_t> tev;   // 3 per timed call
    int64_t timed_calls = 0;
    double acc_attn_ms = 0, acc_merge_ms = 0;
    int64_t acc_calls = 0;
    std::string err;
};

namespace {

int32_t fail(ets_ctx* c, int32_t code, const std::string& msg) {
    if (c) c->err = msg;
    return code;
}

int32_t cuda_fail(ets_ctx* c, cudaError_t e, const char* what) {
    return fail(c, ETS_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

#define ETS_CUDA(ctx, call)                                        \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call); \
    } while (0)

BlobOffsets pack_offsets(const ets_ctx* c, const ets::Tree& t) {
    BlobOffsets b{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
    b.units = take(t.unit.size() * 4);
    b.items = take(t.items.size() * sizeof(ets::Item));
    b.node_page_off = take(t.node_page_off.size() * 4);
    b.page_ids = take(t.page_ids.size() * 4);
    b.node_leaves = take(t.node_leaves.size() * 4);
    b.leaf_node = take(t.leaf_node.size() * 4);
    b.leaf_slot_off = take(t.leaf_slot_off.size() * 4);
    b.leaf_slots = take(t.leaf_slots.size() * 4);
    b.len_stride = t.n_nodes > 0 ? t.n_nodes : 1;
    b.node_len = take((size_t)c->cfg.num_layers * b.len_stride * 4);
    b.total = off;
    return b;
}

void pack_blob(const ets_ctx* c, const ets::Tree& t, const BlobOffsets& b, char* dst) {
    auto put = [&](size_t off, const void* src, size_t bytes) { if (bytes) std::memcpy(dst + off, src, bytes); };
    put(b.units, t.unit.data(), t.unit.size() * 4);
    put(b.items, t.items.data(), t.items.size() * sizeof(ets::Item));
    put(b.node_page_off, t.node_page_off.data(), t.node_page_off.size() * 4);
    put(b.page_ids, t.page_ids.data(), t.page_ids.size() * 4);
    put(b.node_leaves, t.node_leaves.data(), t.node_leaves.size() * 4);
    put(b.leaf_node, t.leaf_node.data(), t.leaf_node.size() * 4);
    put(b.leaf_slot_off, t.leaf_slot_off.data(), t.leaf_slot_off.size() * 4);
    put(b.leaf_slots, t.leaf_slots.data(), t.leaf_slots.size() * 4);
    for (int l = 0; l < c->cfg.num_layers; ++l)
        put(b.node_len + (size_t)l * b.len_stride * 4, t.len[l].data(), t.len[l].size() * 4);
}

template <typename T>
const T* blob_ptr(const ets_ctx* c, size_t off) { return reinterpret_cast<const T*>(c->ws + c->lay.blob + off); }

}  // namespace

extern "C" {

static int32_t host_join(ets_ctx* c, cudaStream_t s);

// all starts to "never", all ends and counters to zero (synchronises the device: only used around measurements)
static int32_t stamps_clear(ets_ctx* c) {
    char* base = c->ws + c->lay.stamps;
    ETS_CUDA(c, cudaDeviceSynchronize());
    ETS_CUDA(c, cudaMemset(base, 0, sizeof(ets::Stamps)));
    ETS_CUDA(c, cudaMemset(base + offsetof(ets::Stamps, start_ns), 0xFF, sizeof(((ets::Stamps*)nullptr)->start_ns)));
    return ETS_OK;
}

const char* ets_version(void) { return "ets-b200 0.1"; }

const char* ets_last_error(const ets_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int32_t ets_pool_bytes(const ets_config* cfg, size_t* k_bytes, size_t* v_bytes, size_t* workspace_bytes) {
    std::string why;
    if (!config_ok(cfg, why)) return ETS_ERR_INVALID_ARG;
    if (int32_t rc = config_supported(cfg, why)) return rc;
    // each buffer holds the K and V tiles of every other page (see kv_tile)
    const size_t pool = (size_t)cfg->num_layers * ets::pool_pairs(cfg->pages_per_layer) * cfg->num_kv_heads * 2 *
                        ets::tile_bytes(cfg->head_dim);
    if (k_bytes) *k_bytes = pool;
    if (v_bytes) *v_bytes = pool;
    if (workspace_bytes) *workspace_bytes = make_layout(cfg).total;
    return ETS_OK;
}

int32_t ets_create(const ets_config* cfg, void* k_pool, void* v_pool, void* workspace, ets_ctx** out) {
    if (!out) return ETS_ERR_INVALID_ARG;
    *out = nullptr;
    std::string why;
    if (!config_ok(cfg, why)) return ETS_ERR_INVALID_ARG;
    if (int32_t rc = config_supported(cfg, why)) return rc;
    const bool host_only = cfg->device < 0;
    if (!host_only) {
        if (!k_pool || !v_pool || !workspace) return ETS_ERR_INVALID_ARG;
        if (((uintptr_t)k_pool | (uintptr_t)v_pool | (uintptr_t)workspace) & 1023) return ETS_ERR_INVALID_ARG;
    }
    ets_ctx* c = new (std::nothrow) ets_ctx();
    if (!c) return ETS_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->host_only = host_only;
    c->lay = make_layout(cfg);
    c->k_pool = (char*)k_pool;
    c->v_pool = (char*)v_pool;
    c->ws = (char*)workspace;
    c->layer_pool_bytes = ets::pool_pairs(cfg->pages_per_layer) * cfg->num_kv_heads * 2 * ets::tile_bytes(cfg->head_dim);
    const float sm = cfg->sm_scale != 0.f ? cfg->sm_scale : 1.0f / std::sqrt((float)cfg->head_dim);
    c->scale_log2 = sm * 1.4426950408889634f;
    c->fp.num_kv_heads = cfg->num_kv_heads;
    c->fp.gqa = cfg->num_q_heads / cfg->num_kv_heads;
    c->fp.page_size = cfg->page_size;
    c->fp.num_layers = cfg->num_layers;
    c->fp.max_nodes = cfg->max_nodes;
    c->fp.max_leaves = cfg->max_leaves;
    c->fp.max_path_entries = cfg->max_path_entries;
    c->fp.max_partial_slots = c->lay.max_partial_slots;
    c->fp.max_items = c->lay.max_items;
    c->fp.rows_per_item = 16;
    // the cost model's weights can be overridden for tuning runs
    if (const char* e = std::getenv("ETS_COST_ITEM")) c->fp.cost_item = std::atof(e);
    if (const char* e = std::getenv("ETS_COST_ROWS16")) c->fp.cost_rows16 = std::atof(e);
    if (const char* e = std::getenv("ETS_COST_REREAD")) c->fp.cost_reread = std::atof(e);
    if (const char* e = std::getenv("ETS_TAIL_PAGES")) c->fp.tail_pages = std::atoi(e);
    if (const char* e = std::getenv("ETS_WIDE_PIECE")) c->fp.wide_piece = std::atoi(e);
    if (!host_only) {
        cudaError_t e = cudaSetDevice(cfg->device);
        cudaDeviceProp prop{};
        if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, cfg->device);
        if (e == cudaSuccess) {
            c->sm_count = prop.multiProcessorCount;
            for (int i = 0; i < kStages && e == cudaSuccess; ++i) {
                e = cudaHostAlloc((void**)&c->stage_host[i], c->lay.blob_cap, cudaHostAllocDefault);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->stage_ev[i], cudaEventDisableTiming);
            }
            for (int i = 0; i < kDescSlots && e == cudaSuccess; ++i) {
                e = cudaHostAlloc((void**)&c->desc_host[i], c->lay.desc_slot_bytes, cudaHostAllocDefault);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->desc_ev[i], cudaEventDisableTiming);
            }
            if (e == cudaSuccess) e = cudaHostAlloc((void**)&c->status_host, 64, cudaHostAllocDefault);
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->st_in, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->st_comp, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->st_out, cudaStreamNonBlocking);
            {
                cudaEvent_t* evs[] = {&c->cache_ev, &c->ev_join_comp, &c->ev_join_out, &c->ev_entry, &c->ev_q_in[0], &c->ev_q_in[1], &c->ev_q_free[0], &c->ev_q_free[1],
                                      &c->ev_comp[0], &c->ev_comp[1], &c->ev_out_free[0], &c->ev_out_free[1],
                                      &c->ev_kv_in[0], &c->ev_kv_in[1], &c->ev_kv_free[0], &c->ev_kv_free[1],
                                      &c->ev_g_in[0], &c->ev_g_in[1], &c->ev_g_free[0], &c->ev_g_free[1],
                                      &c->ev_g_comp[0], &c->ev_g_comp[1], &c->ev_g_out[0], &c->ev_g_out[1]};
                for (cudaEvent_t* ev : evs)
                    if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
            }
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaMemset(c->ws + c->lay.status, 0, 1024);
            if (e == cudaSuccess) e = ets::narrow_prepare(cfg->head_dim);
            if (e == cudaSuccess) e = ets::wide_prepare(cfg->head_dim);
        }
        if (e != cudaSuccess) {
            ets_destroy(c);
            return ETS_ERR_CUDA;
        }
    }
    c->fp.n_workers = c->sm_count * ets::kNarrowWarps < kMaxWorkers ? c->sm_count * ets::kNarrowWarps : kMaxWorkers;
    ets::tree_init(c->tree, c->fp, cfg->pages_per_layer);
    *out = c;
    return ETS_OK;
}

int32_t ets_destroy(ets_ctx* c) {
    if (!c) return ETS_ERR_INVALID_ARG;
    if (!c->host_only) {
        cudaSetDevice(c->cfg.device);
        cudaDeviceSynchronize();
        for (int i = 0; i < kStages; ++i) {
            if (c->stage_host[i]) cudaFreeHost(c->stage_host[i]);
            if (c->stage_ev[i]) cudaEventDestroy(c->stage_ev[i]);
        }
        for (int i = 0; i < kDescSlots; ++i) {
            if (c->desc_host[i]) cudaFreeHost(c->desc_host[i]);
            if (c->desc_ev[i]) cudaEventDestroy(c->desc_ev[i]);
        }
        if (c->status_host) cudaFreeHost(c->status_host);
        if (c->side) cudaStreamDestroy(c->side);
        if (c->st_in) cudaStreamDestroy(c->st_in);
        if (c->st_comp) cudaStreamDestroy(c->st_comp);
        if (c->st_out) cudaStreamDestroy(c->st_out);
        {
            cudaEvent_t evs[] = {c->cache_ev, c->ev_join_comp, c->ev_join_out, c->ev_entry, c->ev_q_in[0], c->ev_q_in[1], c->ev_q_free[0], c->ev_q_free[1], c->ev_comp[0],
                                 c->ev_comp[1], c->ev_out_free[0], c->ev_out_free[1], c->ev_kv_in[0], c->ev_kv_in[1],
                                 c->ev_kv_free[0], c->ev_kv_free[1], c->ev_g_in[0], c->ev_g_in[1], c->ev_g_free[0],
                                 c->ev_g_free[1], c->ev_g_comp[0], c->ev_g_comp[1], c->ev_g_out[0], c->ev_g_out[1]};
            for (cudaEvent_t ev : evs)
                if (ev) cudaEventDestroy(ev);
        }
        if (c->ev_fork) cudaEventDestroy(c->ev_fork);
        if (c->ev_join) cudaEventDestroy(c->ev_join);
        for (cudaEvent_t e : c->tev) cudaEventDestroy(e);
    }
    delete c;
    return ETS_OK;
}

int32_t ets_set_option(ets_ctx* c, int32_t key, int64_t value) {
    if (!c) return ETS_ERR_INVALID_ARG;
    switch (key) {
        case ETS_OPT_CHUNK_PAGES:
            if (value < 0 || value > 4096) return fail(c, ETS_ERR_INVALID_ARG, "chunk pages out of range");
            c->opt_chunk_pages = (int32_t)value;
            return ETS_OK;
        case ETS_OPT_KERNEL:
            if (value < 0 || value > 1) return fail(c, ETS_ERR_INVALID_ARG, "unknown kernel selector");
            c->opt_kernel = (int32_t)value;
            return ETS_OK;
        case ETS_OPT_HOST_PIPELINE:
            if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
            c->opt_host_pipeline = value != 0;
            return ETS_OK;
        case ETS_OPT_WIDE:
            if (value < 0 || value > 1 << 20) return fail(c, ETS_ERR_INVALID_ARG, "wide threshold out of range");
            c->opt_wide = (int32_t)value;
            c->opt_wide_set = true;
            return ETS_OK;
        case ETS_OPT_OVERLAP_APPEND:
            c->opt_overlap_append = value != 0;
            return ETS_OK;
        case ETS_OPT_PACKED_INPUTS:
            c->opt_packed_inputs = value != 0;
            return ETS_OK;
        case ETS_OPT_PATH_ITEMS:
            c->opt_path_items = value != 0;
            return ETS_OK;
        case ETS_OPT_LAUNCH_CHAIN:
            c->opt_chain = value != 0;
            return ETS_OK;
        case ETS_OPT_TEST_FIRST_WAIT_POLLS:
            if (value > (int64_t)ets::kWaitPolls) return fail(c, ETS_ERR_INVALID_ARG, "poll limit out of range");
            c->opt_first_wait_polls = value < 0 ? ets::kWaitPolls : (uint32_t)value;
            return ETS_OK;
        case ETS_OPT_TIMING:
            if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
            if (value < 0 || value > 2) return fail(c, ETS_ERR_INVALID_ARG, "timing mode must be 0, 1 or 2");
            c->opt_timing = value == 1;
            if (value == 2 && !c->opt_stamps) {
                ETS_CUDA(c, cudaSetDevice(c->cfg.device));
                if (int32_t rc = stamps_clear(c)) return rc;
            }
            c->opt_stamps = value == 2;
            return ETS_OK;
        default:
            return fail(c, ETS_ERR_INVALID_ARG, "unknown option");
    }
}

int32_t ets_tree_build(ets_ctx* c, int32_t n_nodes, const int32_t* parent, const int32_t* cap_tokens,
                       const int32_t* keep_pages_of, int32_t n_leaves, const int32_t* leaf_node,
                       void* cuda_stream) {
    if (!c) return ETS_ERR_INVALID_ARG;
    ets::FlattenParams fp = c->fp;
    fp.chunk_pages = c->opt_chunk_pages;
    fp.wide_rows = (c->opt_wide > 0 && c->opt_kernel == 0) ? 128 : 0;
    fp.wide_min_rows = c->opt_wide;
    if (c->opt_wide_set) fp.wide_min_work = 0;
    fp.wide_alt_rows = c->opt_wide_set ? 0 : 49;   // see ets_flatten.cpp: where the limit sits when the wide kernel would end last
    fp.path_items = c->opt_path_items;
    // A rebuild of the very tree that is current (same arrays, every node keeping its own pages, same options)
    // changes nothing: tables, pages and lengths, on the host and on the device, already are what it would produce.
    if (c->has_tree && keep_pages_of && n_nodes == c->tree.n_nodes && n_leaves == c->tree.n_leaves && n_nodes >= 0 &&
        n_leaves >= 0 && (n_nodes == 0 || (parent && cap_tokens)) && (n_leaves == 0 || leaf_node) &&
        fp.chunk_pages == c->built.chunk_pages && fp.wide_rows == c->built.wide_rows &&
        fp.wide_min_rows == c->built.wide_min_rows && fp.wide_min_work == c->built.wide_min_work &&
        fp.wide_alt_rows == c->built.wide_alt_rows &&
        fp.path_items == c->built.path_items &&
        std::memcmp(parent, c->tree.parent.data(), (size_t)n_nodes * 4) == 0 &&
        std::memcmp(cap_tokens, c->tree.cap.data(), (size_t)n_nodes * 4) == 0 &&
        std::memcmp(leaf_node, c->tree.leaf_node.data(), (size_t)n_leaves * 4) == 0) {
        bool identity = true;
        for (int32_t i = 0; i < n_nodes && identity; ++i) identity = keep_pages_of[i] == i;
        if (identity) return ETS_OK;
    }
    ets::Tree& next = c->spare;
    std::string err;
    int32_t rc = ets::tree_build(c->tree, fp, n_nodes, parent, cap_tokens, keep_pages_of, n_leaves, leaf_node,
                                 next, err);
    if (rc != ETS_OK) return fail(c, rc, err);
    if ((int64_t)(next.unit.size() / 4) > c->lay.max_units)
        return fail(c, ETS_ERR_POOL_EXHAUSTED, "page slots exceed the workspace bound");
    BlobOffsets bo = pack_offsets(c, next);
    if (bo.total > c->lay.blob_cap) return fail(c, ETS_ERR_POOL_EXHAUSTED, "tables exceed the workspace bound");
    if (!c->host_only) {
        cudaStream_t s = (cudaStream_t)cuda_stream;
        ETS_CUDA(c, cudaSetDevice(c->cfg.device));
        if (int32_t jrc = host_join(c, s)) return jrc;   // pipelined host-buffer calls still read the old tables
        const int i = c->stage_next;
        if (c->stage_used[i]) ETS_CUDA(c, cudaEventSynchronize(c->stage_ev[i]));
        pack_blob(c, next, bo, c->stage_host[i]);
        ETS_CUDA(c, cudaMemcpyAsync(c->ws + c->lay.blob, c->stage_host[i], bo.total, cudaMemcpyHostToDevice, s));
        ETS_CUDA(c, cudaEventRecord(c->stage_ev[i], s));
        c->stage_used[i] = true;
        c->stage_next = (i + 1) % kStages;
    }
    std::swap(c->tree, c->spare);
    c->bo = bo;
    c->has_tree = true;
    c->built = fp;
    return ETS_OK;
}

int32_t ets_tree_export(const ets_ctx* c, ets_tables_host* o) {
    if (!c || !o) return ETS_ERR_INVALID_ARG;
    const ets::Tree& t = c->tree;
    o->n_nodes = t.n_nodes;
    o->n_leaves = t.n_leaves;
    o->n_pages = (int64_t)t.page_ids.size();
    o->n_group = t.node_leaf_off.empty() ? 0 : (int64_t)t.node_leaf_off.back();   // without the path-item extension
    o->n_path = (int64_t)t.leaf_path.size();
    auto cp = [](int32_t* dst, const std::vector<int32_t>& v) { if (dst && !v.empty()) std::memcpy(dst, v.data(), v.size() * 4); };
    cp(o->node_page_off, t.node_page_off);
    cp(o->page_ids, t.page_ids);
    cp(o->node_leaf_off, t.node_leaf_off);
    if (o->node_leaves && o->n_group > 0) std::memcpy(o->node_leaves, t.node_leaves.data(), (size_t)o->n_group * 4);
    cp(o->leaf_path_off, t.leaf_path_off);
    cp(o->leaf_path, t.leaf_path);
    cp(o->leaf_path_pos, t.leaf_path_pos);
    cp(o->node_depth, t.depth);
    if (!t.len.empty()) cp(o->node_len, t.len[0]);
    return ETS_OK;
}

int32_t ets_work_export(const ets_ctx* c, ets_work_host* o) {
    if (!c || !o) return ETS_ERR_INVALID_ARG;
    const ets::Tree& t = c->tree;
    o->n_units = (int64_t)t.unit.size() / 4;
    o->n_items = (int64_t)t.items.size();
    o->n_leaf_slots = (int64_t)t.leaf_slots.size();
    o->n_partial_slots = t.n_partial_slots;
    o->n_workers = (int64_t)t.worker_off.size() - 1;
    if (o->worker_off && !t.worker_off.empty()) std::memcpy(o->worker_off, t.worker_off.data(), t.worker_off.size() * 4);
    if (o->unit && !t.unit.empty()) std::memcpy(o->unit, t.unit.data(), t.unit.size() * 4);
    if (o->item && !t.items.empty()) std::memcpy(o->item, t.items.data(), t.items.size() * sizeof(ets::Item));
    if (o->leaf_slot_off) std::memcpy(o->leaf_slot_off, t.leaf_slot_off.data(), t.leaf_slot_off.size() * 4);
    if (o->leaf_slots && !t.leaf_slots.empty()) std::memcpy(o->leaf_slots, t.leaf_slots.data(), t.leaf_slots.size() * 4);
    return ETS_OK;
}

int32_t ets_get_node_len(const ets_ctx* c, int32_t layer, int32_t* node_len) {
    if (!c || !node_len || layer < 0 || layer >= c->cfg.num_layers) return ETS_ERR_INVALID_ARG;
    const auto& v = c->tree.len[layer];
    if (!v.empty()) std::memcpy(node_len, v.data(), v.size() * 4);
    return ETS_OK;
}

int32_t ets_get_stats(const ets_ctx* c, ets_stats* o) {
    if (!c || !o) return ETS_ERR_INVALID_ARG;
    const ets::Tree& t = c->tree;
    std::memset(o, 0, sizeof(*o));
    o->n_nodes = t.n_nodes;
    o->n_leaves = t.n_leaves;
    std::vector<int64_t> cum((size_t)t.n_nodes, 0);
    for (int32_t i = 0; i < t.n_nodes; ++i) {
        const int32_t len = t.len[0][i];
        o->unique_tokens += len;
        cum[i] = len + (t.parent[i] >= 0 ? cum[t.parent[i]] : 0);
        if (t.node_leaf_off[i + 1] > t.node_leaf_off[i]) o->attended_tokens += len;
    }
    for (int32_t l = 0; l < t.n_leaves; ++l) o->path_tokens += cum[t.leaf_node[l]];
    o->unique_kv_bytes = o->unique_tokens * 2 * c->cfg.num_kv_heads * c->cfg.head_dim * 2;
    o->pages_used = (int64_t)t.page_ids.size();
    o->pages_free = (int64_t)t.free_heap.size();
    o->n_segments = t.n_segments;
    o->n_chunks = t.n_chunks;
    o->n_items = (int64_t)t.items.size();
    o->n_units = (int64_t)t.unit.size() / 4;
    o->n_partial_slots = t.n_partial_slots;
    o->n_narrow_items = t.n_narrow_items;
    return ETS_OK;
}

// Make `s` wait for every host-buffer call issued so far (kernels and copies back).
static int32_t host_join(ets_ctx* c, cudaStream_t s) {
    if (!c->host_pending) return ETS_OK;
    ETS_CUDA(c, cudaEventRecord(c->ev_join_comp, c->st_comp));
    ETS_CUDA(c, cudaEventRecord(c->ev_join_out, c->st_out));
    ETS_CUDA(c, cudaStreamWaitEvent(s, c->ev_join_comp, 0));
    ETS_CUDA(c, cudaStreamWaitEvent(s, c->ev_join_out, 0));
    c->host_pending = false;
    c->host_epoch_open = false;
    return ETS_OK;
}

// Everything an append launch reads, for the current tree and one layer.
static ets::AppendArgs append_args(const ets_ctx* c, int32_t layer, const void* desc_dev, const void* ksrc, const void* vsrc) {
    const ets::Tree& t = c->tree;
    ets::AppendArgs a{};
    a.desc = reinterpret_cast<const int4*>(desc_dev);
    a.k_new = reinterpret_cast<const __nv_bfloat16*>(ksrc);
    a.v_new = reinterpret_cast<const __nv_bfloat16*>(vsrc);
    a.k_pool = c->k_pool + (size_t)layer * c->layer_pool_bytes;
    a.v_pool = c->v_pool + (size_t)layer * c->layer_pool_bytes;
    a.node_page_off = blob_ptr<int32_t>(c, c->bo.node_page_off);
    a.page_ids = blob_ptr<int32_t>(c, c->bo.page_ids);
    a.node_len = const_cast<int32_t*>(blob_ptr<int32_t>(c, c->bo.node_len)) + (size_t)layer * c->bo.len_stride;
    a.status = reinterpret_cast<int32_t*>(c->ws + c->lay.status);
    a.n_nodes = t.n_nodes;
    a.n_pages_total = (int32_t)t.page_ids.size();
    a.pages_per_layer = c->cfg.pages_per_layer;
    a.Hkv = c->cfg.num_kv_heads;
    a.D = c->cfg.head_dim;
    a.overlap = 0;
    a.stamps = c->opt_stamps ? reinterpret_cast<ets::Stamps*>(c->ws + c->lay.stamps) : nullptr;
    return a;
}

static int32_t append_impl(ets_ctx* c, int32_t layer, int32_t n_items, const int32_t* node_id,
                           const int32_t* n_new, const void* k_new, const void* v_new, bool host_src,
                           cudaStream_t s, bool join = true) {
    if (!c) return ETS_ERR_INVALID_ARG;
    if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
    if (!c->has_tree) return fail(c, ETS_ERR_STATE, "no tree built");
    if (layer < 0 || layer >= c->cfg.num_layers || n_items < 0) return fail(c, ETS_ERR_INVALID_ARG, "layer or count");
    if (n_items == 0) return ETS_OK;
    if (!node_id || !n_new || !k_new || !v_new) return fail(c, ETS_ERR_INVALID_ARG, "null array");
    if (((uintptr_t)k_new | (uintptr_t)v_new) & 15) return fail(c, ETS_ERR_INVALID_ARG, "k_new/v_new must be 16-byte aligned");
    if (n_items > c->cfg.max_nodes) return fail(c, ETS_ERR_INVALID_ARG, "more items than nodes");
    ets::Tree& t = c->tree;
    std::vector<int32_t>& len = t.len[layer];
    // validate everything before touching any state
    int64_t total = 0;
    int32_t max_new = 0;
    std::vector<char> seen;
    seen.assign((size_t)t.n_nodes, 0);
    for (int32_t i = 0; i < n_items; ++i) {
        const int32_t v = node_id[i];
        if (v < 0 || v >= t.n_nodes) return fail(c, ETS_ERR_INVALID_ARG, "node_id out of range");
        if (n_new[i] < 0) return fail(c, ETS_ERR_INVALID_ARG, "n_new < 0");
        if (seen[v]) return fail(c, ETS_ERR_INVALID_ARG, "node named twice in one append");
        seen[v] = 1;
        if ((int64_t)len[v] + n_new[i] > t.cap[v]) return fail(c, ETS_ERR_POOL_EXHAUSTED, "append beyond cap_tokens");
        total += n_new[i];
        max_new = n_new[i] > max_new ? n_new[i] : max_new;
    }
    if (host_src && total > c->lay.max_append_tokens)
        return fail(c, ETS_ERR_POOL_EXHAUSTED, "more tokens than max_append_tokens in a host append");
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    const cudaStream_t user = s;
    const int hb = (int)(c->n_host_append & 1u);
    if (!host_src && join) {
        if (int32_t jrc = host_join(c, s)) return jrc;
    }
    if (host_src) {
        // copy in on the library's input stream into the staging area that is free, run the kernel on
        // the library's compute stream; the caller's stream only waits for the result at the end
        const size_t bytes = (size_t)total * c->cfg.num_kv_heads * c->cfg.head_dim * 2;
        if (!c->host_epoch_open) {
            ETS_CUDA(c, cudaEventRecord(c->ev_entry, user));
            ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_entry, 0));
            ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_entry, 0));
            c->host_epoch_open = c->opt_host_pipeline;
        }
        if (c->kv_used[hb]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_kv_free[hb], 0));
        ETS_CUDA(c, cudaMemcpyAsync(c->ws + c->lay.k_stage + hb * c->lay.kv_stride, k_new, bytes, cudaMemcpyHostToDevice, c->st_in));
        ETS_CUDA(c, cudaMemcpyAsync(c->ws + c->lay.v_stage + hb * c->lay.kv_stride, v_new, bytes, cudaMemcpyHostToDevice, c->st_in));
        ETS_CUDA(c, cudaEventRecord(c->ev_kv_in[hb], c->st_in));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_kv_in[hb], 0));
        s = c->st_comp;
    }
    char* desc_dev = nullptr;
    const bool cacheable = max_new <= 8;   // one block per item: the kernel may read the start itself
    const bool hit = cacheable && c->cache_valid && (int32_t)c->cache_nodes.size() == n_items &&
                     std::memcmp(c->cache_nodes.data(), node_id, (size_t)n_items * 4) == 0 &&
                     std::memcmp(c->cache_nnew.data(), n_new, (size_t)n_items * 4) == 0;
    if (hit) {
        desc_dev = c->ws + c->lay.desc + (size_t)kDescSlots * c->lay.desc_slot_bytes;
        if (c->cache_stream != s) {   // the list was uploaded on another stream: order after it
            ETS_CUDA(c, cudaStreamWaitEvent(s, c->cache_ev, 0));
        }
    } else {
        const int slot = c->desc_next;
        if (c->desc_used[slot]) ETS_CUDA(c, cudaEventSynchronize(c->desc_ev[slot]));
        int4* d = c->desc_host[slot];
        int32_t src = 0;
        for (int32_t i = 0; i < n_items; ++i) {
            d[i] = make_int4(node_id[i], cacheable ? -1 : len[node_id[i]], n_new[i], src);
            src += n_new[i];
        }
        const int dev_slot = cacheable ? kDescSlots : slot;
        desc_dev = c->ws + c->lay.desc + (size_t)dev_slot * c->lay.desc_slot_bytes;
        if (cacheable && c->cache_valid && c->cache_stream != s) {
            // a kernel on the other stream may still read the cached list we are about to replace
            ETS_CUDA(c, cudaEventRecord(c->cache_ev, c->cache_stream));
            ETS_CUDA(c, cudaStreamWaitEvent(s, c->cache_ev, 0));
        }
        ETS_CUDA(c, cudaMemcpyAsync(desc_dev, d, (size_t)n_items * 16, cudaMemcpyHostToDevice, s));
        ETS_CUDA(c, cudaEventRecord(c->desc_ev[slot], s));
        c->desc_used[slot] = true;
        c->desc_next = (slot + 1) % kDescSlots;
        if (cacheable) {
            ETS_CUDA(c, cudaEventRecord(c->cache_ev, s));
            c->cache_nodes.assign(node_id, node_id + n_items);
            c->cache_nnew.assign(n_new, n_new + n_items);
            c->cache_valid = true;
            c->cache_stream = s;
        }
    }
    const void* ksrc = k_new;
    const void* vsrc = v_new;
    if (host_src) {
        ksrc = c->ws + c->lay.k_stage + hb * c->lay.kv_stride;
        vsrc = c->ws + c->lay.v_stage + hb * c->lay.kv_stride;
    }
    ets::AppendArgs a = append_args(c, layer, desc_dev, ksrc, vsrc);
    a.overlap = (c->opt_chain && c->opt_overlap_append && !host_src) ? 1 : 0;
    ets::launch_kv_append(a, n_items, max_new, c->opt_chain, s);
    ETS_CUDA(c, cudaGetLastError());
    if (host_src) {
        ETS_CUDA(c, cudaEventRecord(c->ev_kv_free[hb], c->st_comp));
        if (c->opt_host_pipeline) c->host_pending = true;
        else ETS_CUDA(c, cudaStreamWaitEvent(user, c->ev_kv_free[hb], 0));   // the caller's stream sees the append
        c->kv_used[hb] = true;
        ++c->n_host_append;
    }
    for (int32_t i = 0; i < n_items; ++i) len[node_id[i]] += n_new[i];
    return ETS_OK;
}

int32_t ets_kv_append(ets_ctx* c, int32_t layer, int32_t n_items, const int32_t* node_id, const int32_t* n_new,
                      const void* k_new, const void* v_new, void* cuda_stream) {
    return append_impl(c, layer, n_items, node_id, n_new, k_new, v_new, false, (cudaStream_t)cuda_stream);
}

int32_t ets_kv_append_host(ets_ctx* c, int32_t layer, int32_t n_items, const int32_t* node_id,
                           const int32_t* n_new, const void* k_new, const void* v_new, void* cuda_stream) {
    return append_impl(c, layer, n_items, node_id, n_new, k_new, v_new, true, (cudaStream_t)cuda_stream);
}

// The node-partial attention launches for the current tree: wide query groups on the tcgen05
// kernel, everything else on the narrow kernel (or all of it on the scalar kernel when selected).
static int32_t launch_attention(ets_ctx* c, const ets::DecodeArgs& a, cudaStream_t s) {
    const int D = c->cfg.head_dim;
    const int n_narrow = c->tree.n_narrow_items;
    const int n_wide = (int)c->tree.items.size() - n_narrow;
    if (c->opt_kernel == 1) {
        if (n_wide > 0) return fail(c, ETS_ERR_STATE, "rebuild the tree after changing ETS_OPT_KERNEL");
        ets::launch_partial_fma(a, D, a.n_items, s);
        return ETS_OK;
    }
    // one CTA per SM; fewer when there are fewer narrow items than resident warps
    const int n_ctas = std::min((c->fp.n_workers + ets::kNarrowWarps - 1) / ets::kNarrowWarps,
                                (n_narrow + ets::kNarrowWarps - 1) / ets::kNarrowWarps);
    const bool chain = c->opt_chain;
    if (n_wide > 0 && n_narrow > 0 && chain) {
        // The two kernels write disjoint partial slots and are sized to share an SM.  Both go to the caller's
        // stream, the wide one as the programmatic dependent of the narrow one: it starts as soon as every
        // CTA of the narrow kernel (one per SM, all resident at once) has passed its wait for the kernels
        // ahead, runs beside it, and its last CTA waits for the narrow kernel before it leaves, so whatever
        // follows in the stream is ordered behind both.
        ets::DecodeArgs aw = a;
        aw.wide_behind_narrow = 1;
        ets::launch_partial_narrow(a, D, n_ctas, true, s);
        ets::launch_partial_wide(aw, D, n_narrow, n_wide, true, s);
    } else if (n_wide > 0 && n_narrow > 0) {
        // ordinary launches: the wide kernel runs on a second stream, forked from and joined back into
        // the caller's stream
        ETS_CUDA(c, cudaEventRecord(c->ev_fork, s));
        ETS_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_fork, 0));
        ets::launch_partial_narrow(a, D, n_ctas, false, s);
        ets::launch_partial_wide(a, D, n_narrow, n_wide, false, c->side);
        ETS_CUDA(c, cudaEventRecord(c->ev_join, c->side));
        ETS_CUDA(c, cudaStreamWaitEvent(s, c->ev_join, 0));
    } else if (n_wide > 0) {
        ets::launch_partial_wide(a, D, n_narrow, n_wide, chain, s);
    } else if (n_narrow > 0) {
        ets::launch_partial_narrow(a, D, n_ctas, chain, s);
    }
    return ETS_OK;
}

// Everything a decode launch reads, for the current tree and one layer.
static ets::DecodeArgs decode_args(const ets_ctx* c, int32_t layer, const void* q, void* out, float* lse,
                                   float2* part_ml, float* part_o) {
    const ets::Tree& t = c->tree;
    ets::DecodeArgs a{};
    a.units = blob_ptr<int4>(c, c->bo.units);
    a.items = blob_ptr<ets::DevItem>(c, c->bo.items);
    a.node_leaves = blob_ptr<int32_t>(c, c->bo.node_leaves);
    a.node_len = blob_ptr<int32_t>(c, c->bo.node_len) + (size_t)layer * c->bo.len_stride;
    a.leaf_node = blob_ptr<int32_t>(c, c->bo.leaf_node);
    a.leaf_limit = nullptr;
    a.leaf_slot_off = blob_ptr<int32_t>(c, c->bo.leaf_slot_off);
    a.leaf_slots = blob_ptr<int32_t>(c, c->bo.leaf_slots);
    a.q = reinterpret_cast<const __nv_bfloat16*>(q);
    a.out = reinterpret_cast<__nv_bfloat16*>(out);
    a.lse = lse;
    a.k_pool = c->k_pool + (size_t)layer * c->layer_pool_bytes;
    a.v_pool = c->v_pool + (size_t)layer * c->layer_pool_bytes;
    a.part_ml = part_ml;
    a.part_o = part_o;
    a.status = reinterpret_cast<int32_t*>(c->ws + c->lay.status);
    a.queue = a.status + 16;   // the status area is 1 KiB, zeroed at creation; the kernel rewinds the queue itself
    a.n_items = (int32_t)t.items.size();
    a.n_narrow = t.n_narrow_items;
    a.n_leaves = t.n_leaves;
    a.n_units = (int32_t)(t.unit.size() / 4);
    a.Hq = c->cfg.num_q_heads;
    a.Hkv = c->cfg.num_kv_heads;
    a.G = c->cfg.num_q_heads / c->cfg.num_kv_heads;
    a.pages_per_layer = c->cfg.pages_per_layer;
    a.scale_log2 = c->scale_log2;
    a.first_wait_polls = c->opt_first_wait_polls;
    a.wide_behind_narrow = 0;
    a.stamps = c->opt_stamps ? reinterpret_cast<ets::Stamps*>(c->ws + c->lay.stamps) : nullptr;
    return a;
}

static int32_t decode_impl(ets_ctx* c, int32_t layer, const void* q, void* out, float* lse, cudaStream_t s) {
    const ets::Tree& t = c->tree;
    if (t.n_leaves == 0) return ETS_OK;
    const ets::DecodeArgs a = decode_args(c, layer, q, out, lse, reinterpret_cast<float2*>(c->ws + c->lay.part_ml),
                                          reinterpret_cast<float*>(c->ws + c->lay.part_o));

    cudaEvent_t* ev = nullptr;
    if (c->opt_timing) {
        if (c->timed_calls >= kTimingCap) {  // drain so that the pool can be reused
            double x, y; int64_t n;
            ets_timing_read(c, &x, &y, &n);
            c->acc_attn_ms += x; c->acc_merge_ms += y; c->acc_calls += n;
        }
        while ((int64_t)c->tev.size() < 3 * (c->timed_calls + 1)) {
            cudaEvent_t e;
            ETS_CUDA(c, cudaEventCreate(&e));
            c->tev.push_back(e);
        }
        ev = &c->tev[3 * c->timed_calls];
        ETS_CUDA(c, cudaEventRecord(ev[0], s));
    }
    if (int32_t rc = launch_attention(c, a, s)) return rc;
    if (ev) ETS_CUDA(c, cudaEventRecord(ev[1], s));
    ets::launch_merge(a, c->cfg.head_dim, c->opt_chain, s);
    if (ev) {
        ETS_CUDA(c, cudaEventRecord(ev[2], s));
        c->timed_calls++;
    }
    ETS_CUDA(c, cudaGetLastError());
    return ETS_OK;
}

static int32_t decode_check(ets_ctx* c, int32_t layer, const void* q, void* out, bool prefill = false) {
    if (!c) return ETS_ERR_INVALID_ARG;
    if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
    if (!c->has_tree) return fail(c, ETS_ERR_STATE, "no tree built");
    if (c->tree.path_items && !prefill) return fail(c, ETS_ERR_STATE, "the tree was built with ETS_OPT_PATH_ITEMS: prefill only");
    if (layer < 0 || layer >= c->cfg.num_layers) return fail(c, ETS_ERR_INVALID_ARG, "layer out of range");
    if (c->tree.n_leaves > 0 && (!q || !out)) return fail(c, ETS_ERR_INVALID_ARG, "null q or out");
    return ETS_OK;
}

int32_t ets_tree_attn_decode(ets_ctx* c, int32_t layer, const void* q, void* out, float* lse, void* cuda_stream) {
    if (int32_t rc = decode_check(c, layer, q, out)) return rc;
    if (((uintptr_t)q | (uintptr_t)out) & 15) return fail(c, ETS_ERR_INVALID_ARG, "q/out must be 16-byte aligned");
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    if (int32_t jrc = host_join(c, (cudaStream_t)cuda_stream)) return jrc;
    return decode_impl(c, layer, q, out, lse, (cudaStream_t)cuda_stream);
}

int32_t ets_decode_step(ets_ctx* c, int32_t layer, const void* k_new, const void* v_new, const void* q, void* out,
                        float* lse, void* cuda_stream) {
    if (int32_t rc = decode_check(c, layer, q, out)) return rc;
    if (((uintptr_t)q | (uintptr_t)out) & 15) return fail(c, ETS_ERR_INVALID_ARG, "q/out must be 16-byte aligned");
    const ets::Tree& t = c->tree;
    if (t.n_leaves == 0) return ETS_OK;
    if ((int32_t)c->step_ones.size() != t.n_leaves) c->step_ones.assign((size_t)t.n_leaves, 1);
    // the token of leaf l goes to leaf_node[l]; the append refuses a node that two leaves sit at
    if (int32_t rc = append_impl(c, layer, t.n_leaves, t.leaf_node.data(), c->step_ones.data(), k_new, v_new, false,
                                 (cudaStream_t)cuda_stream))
        return rc;
    return decode_impl(c, layer, q, out, lse, (cudaStream_t)cuda_stream);
}

int32_t ets_tree_attn_prefill(ets_ctx* c, int32_t layer, const void* q, const int32_t* leaf_limit, void* out, float* lse,
                              void* cuda_stream) {
    if (int32_t rc = decode_check(c, layer, q, out, true)) return rc;
    if (((uintptr_t)q | (uintptr_t)out) & 15) return fail(c, ETS_ERR_INVALID_ARG, "q/out must be 16-byte aligned");
    if (c->tree.n_leaves > 0 && !leaf_limit) return fail(c, ETS_ERR_INVALID_ARG, "null leaf_limit");
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (int32_t jrc = host_join(c, s)) return jrc;
    const ets::Tree& t = c->tree;
    if (t.n_leaves == 0) return ETS_OK;
    ets::DecodeArgs a = decode_args(c, layer, q, out, lse, reinterpret_cast<float2*>(c->ws + c->lay.part_ml),
                                    reinterpret_cast<float*>(c->ws + c->lay.part_o));
    a.leaf_limit = leaf_limit;
    // Query groups of more than 16 rows are dense contractions and run on the tcgen05 kernel; the few
    // items of smaller groups (steps of a handful of tokens) take the scalar kernel, which knows the limit too.
    const int D = c->cfg.head_dim;
    const int n_narrow = t.n_narrow_items, n_wide = (int)t.items.size() - n_narrow;
    ets::launch_partial_fma(a, D, n_narrow, s);
    ets::launch_partial_wide(a, D, n_narrow, n_wide, false, s);
    ets::launch_merge(a, D, false, s);
    ETS_CUDA(c, cudaGetLastError());
    return ETS_OK;
}

int32_t ets_tree_attn_decode_host(ets_ctx* c, int32_t layer, const void* q, void* out, float* lse,
                                  void* cuda_stream) {
    if (int32_t rc = decode_check(c, layer, q, out)) return rc;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    const size_t rows = (size_t)c->tree.n_leaves * c->cfg.num_q_heads;
    const size_t qbytes = rows * c->cfg.head_dim * 2;
    if (rows == 0) return ETS_OK;
    // Three library streams: q goes in on one, the kernels run on the second, out/lse come back on the
    // third; the staging areas alternate between calls, so the copies of one call overlap the kernels of
    // the next.  The caller's stream waits for this call's copy-out, which keeps the contract that the
    // results are valid once that stream has passed the call.
    const int hb = (int)(c->n_host_decode & 1u);
    char* qd = c->ws + c->lay.q_stage + hb * c->lay.q_stride;
    char* od = c->ws + c->lay.out_stage + hb * c->lay.q_stride;
    float* ld = reinterpret_cast<float*>(c->ws + c->lay.lse_stage + hb * c->lay.lse_stride);
    if (!c->host_epoch_open) {
        ETS_CUDA(c, cudaEventRecord(c->ev_entry, s));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_entry, 0));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_entry, 0));
        c->host_epoch_open = c->opt_host_pipeline;
    }
    if (c->q_used[hb]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_q_free[hb], 0));
    ETS_CUDA(c, cudaMemcpyAsync(qd, q, qbytes, cudaMemcpyHostToDevice, c->st_in));
    ETS_CUDA(c, cudaEventRecord(c->ev_q_in[hb], c->st_in));
    ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_q_in[hb], 0));
    if (c->out_used[hb]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_out_free[hb], 0));
    if (int32_t rc = decode_impl(c, layer, qd, od, lse ? ld : nullptr, c->st_comp)) return rc;
    ETS_CUDA(c, cudaEventRecord(c->ev_q_free[hb], c->st_comp));   // kernels done: q staging reusable, out ready
    ETS_CUDA(c, cudaStreamWaitEvent(c->st_out, c->ev_q_free[hb], 0));
    ETS_CUDA(c, cudaMemcpyAsync(out, od, qbytes, cudaMemcpyDeviceToHost, c->st_out));
    if (lse) ETS_CUDA(c, cudaMemcpyAsync(lse, ld, rows * 4, cudaMemcpyDeviceToHost, c->st_out));
    ETS_CUDA(c, cudaEventRecord(c->ev_out_free[hb], c->st_out));
    if (c->opt_host_pipeline) c->host_pending = true;
    else ETS_CUDA(c, cudaStreamWaitEvent(s, c->ev_out_free[hb], 0));
    c->q_used[hb] = c->out_used[hb] = true;
    ++c->n_host_decode;
    return ETS_OK;
}

int32_t ets_note_decode_steps(ets_ctx* c, int32_t layer, int32_t times) {
    if (!c) return ETS_ERR_INVALID_ARG;
    if (!c->has_tree) return fail(c, ETS_ERR_STATE, "no tree built");
    if (layer < 0 || layer >= c->cfg.num_layers || times < 0) return fail(c, ETS_ERR_INVALID_ARG, "layer or count");
    ets::Tree& t = c->tree;
    std::vector<int32_t>& len = t.len[layer];
    std::vector<int32_t> add((size_t)t.n_nodes, 0);
    for (int32_t l = 0; l < t.n_leaves; ++l) add[t.leaf_node[l]] += times;
    for (int32_t v = 0; v < t.n_nodes; ++v)
        if ((int64_t)len[v] + add[v] > t.cap[v]) return fail(c, ETS_ERR_POOL_EXHAUSTED, "the replayed steps ran beyond cap_tokens");
    for (int32_t v = 0; v < t.n_nodes; ++v) len[v] += add[v];
    return ETS_OK;
}

int32_t ets_decode_step_host(ets_ctx* c, int32_t layer, const void* k_new, const void* v_new, const void* q, void* out,
                             float* lse, void* cuda_stream) {
    if (int32_t rc = decode_check(c, layer, q, out)) return rc;
    if (!k_new || !v_new) return fail(c, ETS_ERR_INVALID_ARG, "null k_new or v_new");
    ets::Tree& t = c->tree;
    if (t.n_leaves == 0) return ETS_OK;
    if ((int32_t)c->step_ones.size() != t.n_leaves) c->step_ones.assign((size_t)t.n_leaves, 1);
    // The short way needs the append's descriptor list (leaf_node, all ones) to be the one already on the
    // device for the library's compute stream; otherwise take the two calls, which put it there.
    const bool fast = c->cache_valid && c->cache_stream == c->st_comp && (int32_t)c->cache_nodes.size() == t.n_leaves &&
                      std::memcmp(c->cache_nodes.data(), t.leaf_node.data(), (size_t)t.n_leaves * 4) == 0 &&
                      std::memcmp(c->cache_nnew.data(), c->step_ones.data(), (size_t)t.n_leaves * 4) == 0 &&
                      t.n_leaves <= c->lay.max_append_tokens;
    if (!fast) {
        if (int32_t rc = append_impl(c, layer, t.n_leaves, t.leaf_node.data(), c->step_ones.data(), k_new, v_new, true,
                                     (cudaStream_t)cuda_stream))
            return rc;
        return ets_tree_attn_decode_host(c, layer, q, out, lse, cuda_stream);
    }
    std::vector<int32_t>& len = t.len[layer];
    for (int32_t l = 0; l < t.n_leaves; ++l)   // the cached list has distinct nodes; only capacity can fail
        if (len[t.leaf_node[l]] + 1 > t.cap[t.leaf_node[l]]) return fail(c, ETS_ERR_POOL_EXHAUSTED, "append beyond cap_tokens");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    const size_t rows = (size_t)t.n_leaves * c->cfg.num_q_heads;
    const size_t qbytes = rows * c->cfg.head_dim * 2;
    const size_t kvbytes = (size_t)t.n_leaves * c->cfg.num_kv_heads * c->cfg.head_dim * 2;
    const int hb = (int)(c->n_host_decode & 1u), hk = (int)(c->n_host_append & 1u);
    char* kd = c->ws + c->lay.k_stage + hk * c->lay.kv_stride;
    char* vd = c->ws + c->lay.v_stage + hk * c->lay.kv_stride;
    char* qd = c->ws + c->lay.q_stage + hb * c->lay.q_stride;
    // A fused projection leaves k, v and q of a layer next to each other; then one copy brings all three
    // (a host-to-device copy of half a megabyte costs about as much in set-up as in transfer).  Adjacent
    // addresses alone do not prove one allocation (two pinned blocks can touch, and a copy may not span
    // them), so the caller has to promise it.
    const bool packed = c->opt_packed_inputs && (const char*)v_new == (const char*)k_new + kvbytes && (const char*)q == (const char*)v_new + kvbytes;
    if (packed) {
        kd = c->ws + c->lay.pk_stage + hb * c->lay.pk_stride;   // guarded by the same events as the q area
        vd = kd + kvbytes;
        qd = vd + kvbytes;
    }
    char* od = c->ws + c->lay.out_stage + hb * c->lay.q_stride;
    float* ld = reinterpret_cast<float*>(c->ws + c->lay.lse_stage + hb * c->lay.lse_stride);
    if (!c->host_epoch_open) {
        ETS_CUDA(c, cudaEventRecord(c->ev_entry, s));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_entry, 0));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_entry, 0));
        c->host_epoch_open = c->opt_host_pipeline;
    }
    // all three inputs go in on one stream and are announced by one event
    if (c->kv_used[hk]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_kv_free[hk], 0));
    if (c->q_used[hb]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_q_free[hb], 0));
    if (packed) {
        ETS_CUDA(c, cudaMemcpyAsync(kd, k_new, 2 * kvbytes + qbytes, cudaMemcpyHostToDevice, c->st_in));
    } else {
        ETS_CUDA(c, cudaMemcpyAsync(kd, k_new, kvbytes, cudaMemcpyHostToDevice, c->st_in));
        ETS_CUDA(c, cudaMemcpyAsync(vd, v_new, kvbytes, cudaMemcpyHostToDevice, c->st_in));
        ETS_CUDA(c, cudaMemcpyAsync(qd, q, qbytes, cudaMemcpyHostToDevice, c->st_in));
    }
    ETS_CUDA(c, cudaEventRecord(c->ev_q_in[hb], c->st_in));
    ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_q_in[hb], 0));
    if (c->out_used[hb]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_out_free[hb], 0));
    const char* desc_dev = c->ws + c->lay.desc + (size_t)kDescSlots * c->lay.desc_slot_bytes;
    ets::launch_kv_append(append_args(c, layer, desc_dev, kd, vd), t.n_leaves, 1, c->opt_chain, c->st_comp);
    if (int32_t rc = decode_impl(c, layer, qd, od, lse ? ld : nullptr, c->st_comp)) return rc;
    ETS_CUDA(c, cudaEventRecord(c->ev_q_free[hb], c->st_comp));    // kernels done: the q and k/v staging is reusable, out is ready
    ETS_CUDA(c, cudaEventRecord(c->ev_kv_free[hk], c->st_comp));
    ETS_CUDA(c, cudaStreamWaitEvent(c->st_out, c->ev_q_free[hb], 0));
    ETS_CUDA(c, cudaMemcpyAsync(out, od, qbytes, cudaMemcpyDeviceToHost, c->st_out));
    if (lse) ETS_CUDA(c, cudaMemcpyAsync(lse, ld, rows * 4, cudaMemcpyDeviceToHost, c->st_out));
    ETS_CUDA(c, cudaEventRecord(c->ev_out_free[hb], c->st_out));
    if (c->opt_host_pipeline) c->host_pending = true;
    else ETS_CUDA(c, cudaStreamWaitEvent(s, c->ev_out_free[hb], 0));
    c->q_used[hb] = c->out_used[hb] = c->kv_used[hk] = true;
    ++c->n_host_decode;
    ++c->n_host_append;
    for (int32_t l = 0; l < t.n_leaves; ++l) len[t.leaf_node[l]] += 1;
    return ETS_OK;
}

// A decode step of several consecutive layers from host buffers.  A host-to-device copy of a few MiB runs at half
// the rate of one of tens of MiB, so the inputs of kGroupLayers layers travel in one copy, the layers' kernels run
// back to back on the compute stream, and their outputs come back in one copy; groups alternate between two
// staging areas, so the copies of one group overlap the kernels of its neighbours.
int32_t ets_decode_step_host_layers(ets_ctx* c, int32_t first_layer, int32_t n_layers, const void* inputs, void* out,
                                    float* lse, void* cuda_stream) {
    if (n_layers <= 0) return c ? fail(c, ETS_ERR_INVALID_ARG, "n_layers must be positive") : ETS_ERR_INVALID_ARG;
    if (int32_t rc = decode_check(c, first_layer, inputs, out)) return rc;
    if (int32_t rc = decode_check(c, first_layer + n_layers - 1, inputs, out)) return rc;
    ets::Tree& t = c->tree;
    if (t.n_leaves == 0) return ETS_OK;
    if (t.n_leaves > c->lay.max_append_tokens) return fail(c, ETS_ERR_POOL_EXHAUSTED, "more leaves than max_append_tokens");
    if ((int32_t)c->step_ones.size() != t.n_leaves) c->step_ones.assign((size_t)t.n_leaves, 1);
    {   // everything that can fail is checked before the first launch: distinct leaf nodes, room in every layer
        std::vector<char> seen((size_t)t.n_nodes, 0);
        for (int32_t l = 0; l < t.n_leaves; ++l) {
            if (seen[t.leaf_node[l]]) return fail(c, ETS_ERR_INVALID_ARG, "node named twice in one append");
            seen[t.leaf_node[l]] = 1;
        }
        for (int32_t j = 0; j < n_layers; ++j) {
            const std::vector<int32_t>& len = t.len[first_layer + j];
            for (int32_t l = 0; l < t.n_leaves; ++l)
                if (len[t.leaf_node[l]] + 1 > t.cap[t.leaf_node[l]]) return fail(c, ETS_ERR_POOL_EXHAUSTED, "append beyond cap_tokens");
        }
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    const size_t rows = (size_t)t.n_leaves * c->cfg.num_q_heads;
    const size_t qbytes = rows * c->cfg.head_dim * 2;
    const size_t kvbytes = (size_t)t.n_leaves * c->cfg.num_kv_heads * c->cfg.head_dim * 2;
    const size_t rec = 2 * kvbytes + qbytes;
    if (!c->host_epoch_open) {
        ETS_CUDA(c, cudaEventRecord(c->ev_entry, s));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_entry, 0));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_entry, 0));
        c->host_epoch_open = c->opt_host_pipeline;
    }
    // Group sizes: full groups in the middle, one and two layers at either end, so that the first kernels start
    // after a short copy and the last copy back is a short one (with many layers the ends are what stays exposed).
    std::vector<int32_t> sizes;
    {
        int32_t rem = n_layers;
        const bool ramp = n_layers >= 2 * kGroupLayers;
        if (ramp) { sizes.push_back(1); sizes.push_back(2); rem -= 6; }
        for (; rem > 0; rem -= kGroupLayers) sizes.push_back(std::min(kGroupLayers, rem));
        if (ramp) { sizes.push_back(2); sizes.push_back(1); }
    }
    int last = 0;
    int32_t g0 = 0;
    for (size_t gi = 0; gi < sizes.size(); g0 += sizes[gi], ++gi) {
        const int32_t ng = sizes[gi];
        const int b = (int)(c->n_host_group & 1u);
        char* in_d = c->ws + c->lay.grp_in + (size_t)b * c->lay.grp_in_stride;
        char* out_d = c->ws + c->lay.grp_out + (size_t)b * c->lay.grp_out_stride;
        float* lse_d = reinterpret_cast<float*>(c->ws + c->lay.grp_lse + (size_t)b * c->lay.grp_lse_stride);
        if (c->g_used[b]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_in, c->ev_g_free[b], 0));
        ETS_CUDA(c, cudaMemcpyAsync(in_d, (const char*)inputs + (size_t)g0 * rec, (size_t)ng * rec, cudaMemcpyHostToDevice, c->st_in));
        ETS_CUDA(c, cudaEventRecord(c->ev_g_in[b], c->st_in));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_g_in[b], 0));
        if (c->g_used[b]) ETS_CUDA(c, cudaStreamWaitEvent(c->st_comp, c->ev_g_out[b], 0));
        for (int32_t j = 0; j < ng; ++j) {
            const int32_t layer = first_layer + g0 + j;
            const char* kd = in_d + (size_t)j * rec;
            if (int32_t rc = append_impl(c, layer, t.n_leaves, t.leaf_node.data(), c->step_ones.data(), kd, kd + kvbytes,
                                         false, c->st_comp, false))
                return rc;
            if (int32_t rc = decode_impl(c, layer, kd + 2 * kvbytes, out_d + (size_t)j * qbytes,
                                         lse ? lse_d + (size_t)j * rows : nullptr, c->st_comp))
                return rc;
        }
        ETS_CUDA(c, cudaEventRecord(c->ev_g_free[b], c->st_comp));
        ETS_CUDA(c, cudaEventRecord(c->ev_g_comp[b], c->st_comp));
        ETS_CUDA(c, cudaStreamWaitEvent(c->st_out, c->ev_g_comp[b], 0));
        ETS_CUDA(c, cudaMemcpyAsync((char*)out + (size_t)g0 * qbytes, out_d, (size_t)ng * qbytes, cudaMemcpyDeviceToHost, c->st_out));
        if (lse) ETS_CUDA(c, cudaMemcpyAsync(lse + (size_t)g0 * rows, lse_d, (size_t)ng * rows * 4, cudaMemcpyDeviceToHost, c->st_out));
        ETS_CUDA(c, cudaEventRecord(c->ev_g_out[b], c->st_out));
        c->g_used[b] = true;
        ++c->n_host_group;
        last = b;
    }
    if (c->opt_host_pipeline) c->host_pending = true;
    else ETS_CUDA(c, cudaStreamWaitEvent(s, c->ev_g_out[last], 0));   // st_out runs in order: the last group's copy is the last to finish
    return ETS_OK;
}

// ---------------------------------------------------------------------------------------------
// Decode with built-in scratch, for callers that must not allocate.
//
// Some users of this library cannot create device allocations of their own: a plugin that runs
// inside a host application's fixed memory budget, code that is called while another component
// owns the allocator, or a real-time loop in which cudaMalloc (which may synchronise the whole
// device) is not allowed.  Such callers still hand over q and out, but cannot provide room for
// the partial results that the attention kernel writes and the merge kernel reads.  For them the
// library carries a fixed 8 MiB array in device memory; it exists once per GPU that loads the
// library and stays until the process ends.
//
// The array's name is only meaningful to device code.  Host code must translate it with
// cudaGetSymbolAddress, per device and with that device current; that is done on the first call
// for a device and cached.  That first call therefore performs a runtime query and should be made
// before any stream capture begins.
//
// All calls share the one array and it keeps the previous call's contents.  Nothing in it needs to
// start at zero: every partial slot that the merge kernel reads is written in full by the
// attention kernel of the same call.  Two calls that overlap on the GPU (different streams, or
// two contexts on one device) would overwrite each other's partials: run them one after another.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr size_t kStaticScratchBytes = (size_t)8 << 20;
constexpr int kStaticMaxDevices = 64;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
// device address of the array per device ordinal; contexts on different host threads may race to fill an
// entry, so it is an atomic (every thread would store the same value)
std::atomic<unsigned char*> g_static_scratch_addr[kStaticMaxDevices];
}  // namespace

int32_t ets_tree_attn_decode_static(ets_ctx* c, int32_t layer, const void* q, void* out, float* lse,
                                    void* cuda_stream) {
    if (int32_t rc = decode_check(c, layer, q, out)) return rc;
    if (((uintptr_t)q | (uintptr_t)out) & 15) return fail(c, ETS_ERR_INVALID_ARG, "q/out must be 16-byte aligned");
    const int dev = c->cfg.device;
    if (dev >= kStaticMaxDevices) return fail(c, ETS_ERR_UNSUPPORTED, "device ordinal beyond the built-in scratch table");
    const ets::Tree& t = c->tree;
    const int G = c->cfg.num_q_heads / c->cfg.num_kv_heads;
    const int D = c->cfg.head_dim;
    const size_t rows = (size_t)t.n_partial_slots * G;
    const size_t ml_bytes = align_up(rows * sizeof(float2), 256);   // the o part starts on a 256-byte boundary
    const size_t need = ml_bytes + rows * D * sizeof(float);
    if (need > kStaticScratchBytes)
        return fail(c, ETS_ERR_POOL_EXHAUSTED,
                    "tree needs " + std::to_string(need) + " bytes of partial results; the built-in scratch holds " +
                        std::to_string(kStaticScratchBytes) + " (use ets_tree_attn_decode with a workspace)");
    ETS_CUDA(c, cudaSetDevice(dev));
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // like every device entry point: pipelined host-buffer calls still in flight on the library's streams
    // (they append to the pools and use the same item queue) are joined first
    if (int32_t jrc = host_join(c, s)) return jrc;
    unsigned char* scratch = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        void* p = nullptr;
        ETS_CUDA(c, cudaGetSymbolAddress(&p, g_static_scratch));
        scratch = static_cast<unsigned char*>(p);
        g_static_scratch_addr[dev].store(scratch, std::memory_order_release);
    }
    if (t.n_leaves == 0) return ETS_OK;
    const ets::DecodeArgs a = decode_args(c, layer, q, out, lse, reinterpret_cast<float2*>(scratch),
                                          reinterpret_cast<float*>(scratch + ml_bytes));
    if (int32_t rc = launch_attention(c, a, s)) return rc;
    ets::launch_merge(a, D, c->opt_chain, s);
    ETS_CUDA(c, cudaGetLastError());
    return ETS_OK;
}

int32_t ets_kv_read_debug(ets_ctx* c, int32_t layer, int32_t node, void* k_out, void* v_out, void* cuda_stream) {
    if (!c) return ETS_ERR_INVALID_ARG;
    if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
    if (!c->has_tree) return fail(c, ETS_ERR_STATE, "no tree built");
    if (layer < 0 || layer >= c->cfg.num_layers || node < 0 || node >= c->tree.n_nodes)
        return fail(c, ETS_ERR_INVALID_ARG, "layer or node out of range");
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    const int32_t* pages = blob_ptr<int32_t>(c, c->bo.page_ids) + c->tree.node_page_off[node];
    ets::launch_kv_read(c->k_pool + (size_t)layer * c->layer_pool_bytes,
                        c->v_pool + (size_t)layer * c->layer_pool_bytes, pages, c->tree.len[layer][node],
                        c->cfg.pages_per_layer, c->cfg.num_kv_heads, c->cfg.head_dim, (__nv_bfloat16*)k_out, (__nv_bfloat16*)v_out,
                        (cudaStream_t)cuda_stream);
    ETS_CUDA(c, cudaGetLastError());
    return ETS_OK;
}

int32_t ets_host_join(ets_ctx* c, void* cuda_stream) {
    if (!c) return ETS_ERR_INVALID_ARG;
    if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    return host_join(c, (cudaStream_t)cuda_stream);
}

int32_t ets_timing_read(ets_ctx* c, double* attn_ms, double* merge_ms, int64_t* n_calls) {
    if (!c || !attn_ms || !merge_ms || !n_calls) return ETS_ERR_INVALID_ARG;
    if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
    double a = c->acc_attn_ms, m = c->acc_merge_ms;
    int64_t n = c->acc_calls;
    c->acc_attn_ms = c->acc_merge_ms = 0;
    c->acc_calls = 0;
    for (int64_t i = 0; i < c->timed_calls; ++i) {
        cudaEvent_t* ev = &c->tev[3 * i];
        ETS_CUDA(c, cudaEventSynchronize(ev[2]));
        float x = 0, y = 0;
        ETS_CUDA(c, cudaEventElapsedTime(&x, ev[0], ev[1]));
        ETS_CUDA(c, cudaEventElapsedTime(&y, ev[1], ev[2]));
        a += x; m += y; ++n;
    }
    c->timed_calls = 0;
    *attn_ms = a; *merge_ms = m; *n_calls = n;
    return ETS_OK;
}

int32_t ets_stamps_read(ets_ctx* c, ets_stamps_host* out) {
    if (!c || !out) return ETS_ERR_INVALID_ARG;
    if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
    static_assert(sizeof(ets_stamps_host) == sizeof(ets::Stamps) && ETS_STAMP_LAUNCHES == ets::kStampLaunches &&
                      ETS_STAMP_KINDS == ets::kStampKinds, "stamp tables out of sync");
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    ETS_CUDA(c, cudaDeviceSynchronize());
    ETS_CUDA(c, cudaMemcpy(out, c->ws + c->lay.stamps, sizeof(ets::Stamps), cudaMemcpyDeviceToHost));
    return stamps_clear(c);
}

int32_t ets_poll_status(ets_ctx* c, void* cuda_stream) {
    if (!c) return ETS_ERR_INVALID_ARG;
    if (c->host_only) return fail(c, ETS_ERR_STATE, "host-only context");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    ETS_CUDA(c, cudaSetDevice(c->cfg.device));
    if (int32_t jrc = host_join(c, s)) return jrc;
    ETS_CUDA(c, cudaMemcpyAsync(c->status_host, c->ws + c->lay.status, 4, cudaMemcpyDeviceToHost, s));
    ETS_CUDA(c, cudaMemsetAsync(c->ws + c->lay.status, 0, 4, s));
    ETS_CUDA(c, cudaStreamSynchronize(s));
    const int32_t v = *c->status_host;
    if (v == 0) return ETS_OK;
    if (v == -7) return fail(c, ETS_ERR_DEVICE_TIMEOUT, "a device-side wait ran out");
    return fail(c, ETS_ERR_INVALID_ARG, "a kernel skipped an out-of-range table entry");
}

}  // extern "C"
