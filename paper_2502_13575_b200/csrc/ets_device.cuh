// Device-side declarations shared by the kernels and the API file.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace ets {

// In-page layout of one (page, kv head) tile: 16 tokens x D bf16, stored as the shared-memory
// image that both the tensor-core paths and the scalar path consume, so that one linear bulk
// copy of the tile needs no rearrangement:
//   byte(t, e) = (t/8) * (D/64)*1024          8-token group
//              + (e/64) * 1024                 64-element half of the head dimension
//              + (t%8) * 128                   row inside the 8x128B swizzle atom
//              + (((e%64)/8) ^ (t%8)) * 16     16-byte chunk, XOR-swizzled by the row
//              + (e%8) * 2
// i.e. rows of 128 bytes in 1024-byte atoms with the 128-byte swizzle pattern.
constexpr int kPageTokens = 16;
constexpr int kNarrowWarps = 8;   // independent warp-workers per CTA of the narrow attention kernel

__host__ __device__ inline size_t tile_bytes(int D) { return (size_t)kPageTokens * D * 2; }

__host__ __device__ inline uint32_t tile_offset(int D, int t, int e) {
    uint32_t r = (uint32_t)t & 7u;
    return (uint32_t)(t >> 3) * (uint32_t)(D / 64) * 1024u + (uint32_t)(e >> 6) * 1024u + r * 128u +
           ((((uint32_t)(e & 63) >> 3) ^ r) << 4) + (uint32_t)(e & 7) * 2u;
}

// Where the K tile of a (page, kv head) lives; its V tile follows it directly, so one bulk copy of two
// tiles brings both (half as many copy requests as one per tile).  Pages alternate between the two
// pool buffers the caller provides: even page ids in the first, odd ones in the second, and inside a
// buffer [kv head][page / 2][K tile | V tile].  Pages of a node usually have consecutive ids, so a
// worker that streams one head of a node reads two contiguous runs.
__host__ __device__ inline size_t pool_pairs(int64_t pages_per_layer) { return ((size_t)pages_per_layer + 1) / 2; }
template <typename P>
__host__ __device__ inline P* kv_tile(P* pool_even, P* pool_odd, int64_t pages_per_layer, int page, int head, size_t tb) {
    P* pool = (page & 1) ? pool_odd : pool_even;
    return pool + ((size_t)head * pool_pairs(pages_per_layer) + (size_t)(page >> 1)) * 2 * tb;
}

// Device time stamps (ETS_OPT_TIMING = 2): per kind of kernel and launch, the earliest start and the latest end over
// its CTAs, read from the GPU's global nanosecond timer.  Kinds: 0 append, 1 narrow attention, 2 wide attention,
// 3 merge, 4 the moment the narrow kernel's wait for the kernel ahead returned (start only).  The launch index of a
// kind is a counter that the last CTA (warp, for the narrow kernel) of a launch to finish advances; launches of one
// kind never overlap each other here, so every CTA of a launch reads the same index.  Costs one predicate per kernel
// when switched off (null pointer).
constexpr int kStampKinds = 5;
constexpr int kStampLaunches = 4096;
struct Stamps {
    unsigned int count[8];
    unsigned int done[8];
    unsigned long long start_ns[kStampKinds][kStampLaunches];
    unsigned long long end_ns[kStampKinds][kStampLaunches];
};
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// returns the launch index (or kStampLaunches when the table is full)
__device__ __forceinline__ unsigned int stamp_start(Stamps* s, int kind) {
    const unsigned int i = min(*((volatile unsigned int*)&s->count[kind]), (unsigned int)kStampLaunches);
    if (i < (unsigned int)kStampLaunches) atomicMin(&s->start_ns[kind][i], global_ns());
    return i;
}
__device__ __forceinline__ void stamp_end(Stamps* s, int kind, unsigned int i, unsigned int n_reports) {
    if (i < (unsigned int)kStampLaunches) atomicMax(&s->end_ns[kind][i], global_ns());
    __threadfence();
    if (atomicAdd(&s->done[kind], 1u) == n_reports - 1) {
        s->done[kind] = 0;
        atomicAdd(&s->count[kind], 1u);
    }
}

struct DevItem {
    int32_t unit_begin, unit_count, kv_head, leaf_list_begin;
    int32_t n_leaves_tile, slot_first, segment, reserved;
};

// Everything a decode launch needs; passed by value.
struct DecodeArgs {
    const int4* units;
    const DevItem* items;
    const int32_t* node_leaves;
    const int32_t* node_len;       // this layer's lengths
    const int32_t* leaf_node;      // node each leaf sits at
    const int32_t* leaf_limit;     // nullable: tokens of its own node each leaf's query may see (step prefill)
    const int32_t* leaf_slot_off;  // per (leaf, kv head)
    const int32_t* leaf_slots;
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    float* lse;
    const char* k_pool;            // this layer's pool buffers (see kv_tile: each holds K and V of half the pages)
    const char* v_pool;
    float2* part_ml;               // [slot][G]  (m in log2 units, l); a slot belongs to one kv head
    float* part_o;                 // [slot][G][D]
    int32_t* queue;                // [0] narrow items handed out beyond the first per warp, [1] warps that have finished,
                                   // [2] CTAs of the wide kernel that have finished (each rewound by the last to report)
    int32_t* status;
    int32_t n_items, n_narrow, n_leaves, n_units;   // narrow items come first in `items`
    int32_t Hq, Hkv, G;
    int64_t pages_per_layer;
    float scale_log2;              // sm_scale * log2(e)
    uint32_t first_wait_polls;     // give-up limit of each worker's first wait for data (kWaitPolls unless a test lowers it)
    int32_t wide_behind_narrow;    // wide kernel: launched as the narrow kernel's programmatic dependent (see launch_attention)
    Stamps* stamps;                // nullable: device time stamps
};

constexpr uint32_t kWaitPolls = 1u << 22;   // polls after which a device-side wait gives up

// Programmatic dependent launch (PTX griddepcontrol).  A kernel launched with the programmatic-serialization
// attribute may start while the kernel before it in the stream is still running, once every CTA of that
// kernel has executed pdl_launch_dependents() or exited.  pdl_wait() returns when that kernel has completed
// and its writes are visible; it returns at once in a kernel that was launched the ordinary way.  Rule kept by
// every kernel here that can be launched this way: nothing an earlier kernel writes is read, and nothing an
// earlier kernel reads is written, before pdl_wait(); and every such kernel executes pdl_wait() before it
// ends, so that "this kernel has completed" always implies "everything before it in the stream has".
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

struct AppendArgs {
    const int4* desc;              // per item: node, start, n_new, src token offset
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    char* k_pool;
    char* v_pool;
    const int32_t* node_page_off;
    const int32_t* page_ids;
    int32_t* node_len;
    int32_t* status;
    int32_t n_nodes, n_pages_total;
    int64_t pages_per_layer;
    int32_t Hkv, D;
    int32_t overlap;               // 1: copy first, wait for the preceding kernel at the end (see launch_kv_append)
    Stamps* stamps;                // nullable: device time stamps
};

void launch_kv_append(const AppendArgs& a, int n_items, int max_new, bool chained, cudaStream_t s);
void launch_kv_read(const char* k_pool, const char* v_pool, const int32_t* page_ids_of_node, int n_tokens,
                    int64_t pages_per_layer, int Hkv, int D, __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t s);
void launch_partial_fma(const DecodeArgs& a, int D, int n_items, cudaStream_t s);
void launch_merge(const DecodeArgs& a, int D, bool chained, cudaStream_t s);
size_t narrow_smem_bytes(int D);
cudaError_t narrow_prepare(int D);
void launch_partial_narrow(const DecodeArgs& a, int D, int n_ctas, bool chained, cudaStream_t s);
size_t wide_smem_bytes(int D);
cudaError_t wide_prepare(int D);
void launch_partial_wide(const DecodeArgs& a, int D, int first_item, int n_wide, bool chained, cudaStream_t s);

// launch configuration with or without the programmatic-serialization attribute
struct ChainLaunch {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    ChainLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool chained) {
        cfg.gridDim = grid;
        cfg.blockDim = block;
        cfg.dynamicSmemBytes = smem;
        cfg.stream = s;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = chained ? 1 : 0;
    }
};

}  // namespace ets
