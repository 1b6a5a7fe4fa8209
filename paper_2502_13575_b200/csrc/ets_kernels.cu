// KV append / read-back, the scalar-FMA node-partial attention kernel and the
// log-sum-exp merge kernel.
#include "ets_device.cuh"
#include "ets_merge.cuh"

namespace ets {

// ------------------------------------------------------------------------------------
// KV append: scatter new token rows [token, kv head, D] into (page, slot) tiles.
// One block handles 8 tokens of one item; a thread moves 16-byte chunks.
// ------------------------------------------------------------------------------------
constexpr int kAppendTokPerBlock = 8;

__device__ __forceinline__ void kv_append_block(const AppendArgs& a) {
    const int4 d = a.desc[blockIdx.y];
    const int node = d.x, n_new = d.z, src_off = d.w;
    const int t0 = blockIdx.x * kAppendTokPerBlock;
    if (t0 >= n_new) return;
    if (node < 0 || node >= a.n_nodes) {
        if (threadIdx.x == 0) atomicExch(a.status, -1);
        return;
    }
    // a negative start means "append at the node's current length" (used when one block covers the
    // whole item, so nobody reads the length after it has been advanced); __syncthreads orders the
    // read before thread 0's update at the end
    const int start = d.y >= 0 ? d.y : a.node_len[node];
    __syncthreads();
    const int chunks_per_head = a.D / 8;
    const int chunks_per_tok = a.Hkv * chunks_per_head;
    const int n_tok = min(kAppendTokPerBlock, n_new - t0);
    const size_t tb = tile_bytes(a.D);
    const int page_base = a.node_page_off[node];
    const int page_cnt = a.node_page_off[node + 1] - page_base;
    for (int i = threadIdx.x; i < n_tok * chunks_per_tok; i += blockDim.x) {
        const int t = t0 + i / chunks_per_tok;
        const int ci = i % chunks_per_tok;
        const int h = ci / chunks_per_head;
        const int c = ci % chunks_per_head;
        const int pos = start + t;
        const int pslot = pos / kPageTokens;
        if (pslot >= page_cnt) {  // beyond the node's reserved pages: refuse, flag, keep going
            atomicExch(a.status, -1);
            continue;
        }
        const int page = a.page_ids[page_base + pslot];
        if (page < 0 || (int64_t)page >= a.pages_per_layer) {
            atomicExch(a.status, -1);
            continue;
        }
        const size_t src = ((size_t)(src_off + t) * a.Hkv + h) * a.D + (size_t)c * 8;
        char* dst = kv_tile(a.k_pool, a.v_pool, a.pages_per_layer, page, h, tb) + tile_offset(a.D, pos % kPageTokens, c * 8);
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(a.k_new + src);
        *reinterpret_cast<uint4*>(dst + tb) = *reinterpret_cast<const uint4*>(a.v_new + src);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) a.node_len[node] = start + n_new;
}

// Launched with the programmatic-serialization attribute when the caller chains its launches (see
// pdl_wait in ets_device.cuh).  The kernel behind it (an attention kernel) may begin at once: it reads
// nothing this kernel writes before its own pdl_wait.  Ordinarily this kernel waits for the one before
// it and then copies.  With `overlap` it copies first and waits at the end: an append touches one
// layer's pages and lengths, which the kernel that signalled (the merge kernel of the previous decode
// call, whose attention kernels have completed by then) does not read, and k_new / v_new are complete
// by the caller's promise; the wait at the end keeps completion transitive, so that the attention
// kernel behind this append cannot overwrite partial results the merge kernel is still reading.
__global__ void __launch_bounds__(256) kv_append_kernel(AppendArgs a) {
    unsigned int stamp = 0;
    if (a.stamps && threadIdx.x == 0) stamp = stamp_start(a.stamps, 0);
    pdl_launch_dependents();
    if (!a.overlap) pdl_wait();
    kv_append_block(a);
    if (a.overlap) pdl_wait();
    if (a.stamps) {
        __syncthreads();
        if (threadIdx.x == 0) stamp_end(a.stamps, 0, stamp, gridDim.x * gridDim.y);
    }
}

void launch_kv_append(const AppendArgs& a, int n_items, int max_new, bool chained, cudaStream_t s) {
    if (n_items <= 0 || max_new <= 0) return;
    dim3 grid((max_new + kAppendTokPerBlock - 1) / kAppendTokPerBlock, n_items);
    ChainLaunch l(grid, dim3(256), 0, s, chained);
    cudaLaunchKernelEx(&l.cfg, kv_append_kernel, a);
}

// ------------------------------------------------------------------------------------
// Read one node's rows back in token order (debug / tests).
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) kv_read_kernel(const char* k_pool, const char* v_pool,
                                                      const int32_t* pages, int n_tokens, int64_t pages_per_layer, int Hkv,
                                                      int D, __nv_bfloat16* k_out, __nv_bfloat16* v_out) {
    const int chunks_per_head = D / 8;
    const int chunks_per_tok = Hkv * chunks_per_head;
    const size_t tb = tile_bytes(D);
    const int64_t total = (int64_t)n_tokens * chunks_per_tok;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(i / chunks_per_tok);
        const int ci = (int)(i % chunks_per_tok);
        const int h = ci / chunks_per_head;
        const int c = ci % chunks_per_head;
        const int page = pages[t / kPageTokens];
        const char* src = kv_tile(k_pool, v_pool, pages_per_layer, page, h, tb) + tile_offset(D, t % kPageTokens, c * 8);
        const size_t dst = ((size_t)t * Hkv + h) * D + (size_t)c * 8;
        if (k_out) *reinterpret_cast<uint4*>(k_out + dst) = *reinterpret_cast<const uint4*>(src);
        if (v_out) *reinterpret_cast<uint4*>(v_out + dst) = *reinterpret_cast<const uint4*>(src + tb);
    }
}

void launch_kv_read(const char* k_pool, const char* v_pool, const int32_t* pages, int n_tokens,
                    int64_t pages_per_layer, int Hkv, int D, __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t s) {
    if (n_tokens <= 0) return;
    int64_t total = (int64_t)n_tokens * Hkv * (D / 8);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 4096) blocks = 4096;
    kv_read_kernel<<<blocks, 256, 0, s>>>(k_pool, v_pool, pages, n_tokens, pages_per_layer, Hkv, D, k_out, v_out);
}

// ------------------------------------------------------------------------------------
// Scalar-FMA node-partial attention.  One block per work item, 4 warps; warp w takes page
// slots w, w+4, ... of the chunk.  A lane owns D/32 consecutive features of every row; the
// q.k dot products are finished with warp shuffles.  Scores are kept in log2 units.
// Generic fallback: any group width, any supported head_dim, no tensor cores.
// ------------------------------------------------------------------------------------
constexpr int kFmaWarps = 4;
constexpr int kMaxRows = 16;

template <int D>
__global__ void __launch_bounds__(kFmaWarps * 32) attn_partial_fma_kernel(DecodeArgs a) {
    constexpr int EPL = D / 32;  // features per lane
    __shared__ float sm_m[kFmaWarps][kMaxRows];
    __shared__ float sm_l[kFmaWarps][kMaxRows];
    __shared__ float sm_o[kFmaWarps][kMaxRows][D];

    const DevItem it = a.items[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.G;
    const int rows = it.n_leaves_tile * G;
    const int h = it.kv_head;
    const int e0 = lane * EPL;

    float q[kMaxRows][EPL];
    float o[kMaxRows][EPL];
    float m[kMaxRows], l[kMaxRows];
    int own[kMaxRows], lim[kMaxRows];   // step prefill: node the row's leaf sits at, tokens of it the row may see
#pragma unroll
    for (int r = 0; r < kMaxRows; ++r) {
        m[r] = -INFINITY;
        l[r] = 0.f;
#pragma unroll
        for (int j = 0; j < EPL; ++j) { q[r][j] = 0.f; o[r][j] = 0.f; }
        own[r] = -1;
        lim[r] = 0;
        if (r < rows) {
            const int leaf = a.node_leaves[it.leaf_list_begin + r / G];
            if (a.leaf_limit != nullptr) {
                own[r] = a.leaf_node[leaf];
                lim[r] = a.leaf_limit[leaf];
            }
            const __nv_bfloat16* qp = a.q + ((size_t)leaf * a.Hq + h * G + r % G) * D + e0;
#pragma unroll
            for (int j = 0; j < EPL; ++j) q[r][j] = __bfloat162float(qp[j]);
        }
    }

    const size_t tb = tile_bytes(D);
    for (int u = warp; u < it.unit_count; u += kFmaWarps) {
        const int4 un = a.units[it.unit_begin + u];
        if (un.x < 0 || (int64_t)un.x >= a.pages_per_layer) {
            if (lane == 0) atomicExch(a.status, -1);
            continue;
        }
        int valid = a.node_len[un.y] - un.z;
        valid = valid < 0 ? 0 : (valid > kPageTokens ? kPageTokens : valid);
        const char* kt = kv_tile(a.k_pool, a.v_pool, a.pages_per_layer, un.x, h, tb);
        const char* vt = kt + tb;
        for (int t = 0; t < valid; ++t) {
            const uint32_t off = tile_offset(D, t, e0);
            float kf[EPL], vf[EPL];
            const __nv_bfloat16* kp = reinterpret_cast<const __nv_bfloat16*>(kt + off);
            const __nv_bfloat16* vp = reinterpret_cast<const __nv_bfloat16*>(vt + off);
#pragma unroll
            for (int j = 0; j < EPL; ++j) { kf[j] = __bfloat162float(kp[j]); vf[j] = __bfloat162float(vp[j]); }
#pragma unroll
            for (int r = 0; r < kMaxRows; ++r) {
                if (r < rows && (un.y != own[r] || un.z + t < lim[r])) {
                    float s = 0.f;
#pragma unroll
                    for (int j = 0; j < EPL; ++j) s = fmaf(q[r][j], kf[j], s);
#pragma unroll
                    for (int x = 16; x > 0; x >>= 1) s += __shfl_xor_sync(0xffffffffu, s, x);
                    s *= a.scale_log2;
                    const float mn = fmaxf(m[r], s);
                    const float corr = exp2f(m[r] - mn);
                    const float p = exp2f(s - mn);
                    l[r] = l[r] * corr + p;
#pragma unroll
                    for (int j = 0; j < EPL; ++j) o[r][j] = o[r][j] * corr + p * vf[j];
                    m[r] = mn;
                }
            }
        }
    }

    // combine the four warps' partials
#pragma unroll
    for (int r = 0; r < kMaxRows; ++r) {
        if (r < rows) {
            if (lane == 0) { sm_m[warp][r] = m[r]; sm_l[warp][r] = l[r]; }
#pragma unroll
            for (int j = 0; j < EPL; ++j) sm_o[warp][r][e0 + j] = o[r][j];
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < rows * D; i += blockDim.x) {
        const int r = i / D, e = i % D;
        float ms = -INFINITY;
#pragma unroll
        for (int w = 0; w < kFmaWarps; ++w) ms = fmaxf(ms, sm_m[w][r]);
        float acc = 0.f, ls = 0.f;
#pragma unroll
        for (int w = 0; w < kFmaWarps; ++w) {
            const float wgt = sm_l[w][r] > 0.f ? exp2f(sm_m[w][r] - ms) : 0.f;
            acc += wgt * sm_o[w][r][e];
            ls += wgt * sm_l[w][r];
        }
        const size_t row = (size_t)(it.slot_first + r / G) * G + r % G;
        a.part_o[row * D + e] = acc;
        if (e == 0) a.part_ml[row] = make_float2(ms, ls);
    }
}

void launch_partial_fma(const DecodeArgs& a, int D, int n_items, cudaStream_t s) {
    if (n_items <= 0) return;
    if (D == 128) attn_partial_fma_kernel<128><<<n_items, kFmaWarps * 32, 0, s>>>(a);
    else attn_partial_fma_kernel<64><<<n_items, kFmaWarps * 32, 0, s>>>(a);
}

// ------------------------------------------------------------------------------------
// Log-sum-exp merge along each leaf's path: one warp per (leaf, query head); plenty of warps,
// because each one is a short chain of dependent loads.
// ------------------------------------------------------------------------------------
#ifndef ETS_MERGE_WARPS
#define ETS_MERGE_WARPS 4
#endif
constexpr int kMergeWarps = ETS_MERGE_WARPS;

template <int D, int kEarly>
__global__ void __launch_bounds__(kMergeWarps * 32) lse_merge_kernel(DecodeArgs a) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kMergeWarps + warp;
    const bool active = row < (int64_t)a.n_leaves * a.Hq;
    // Before the wait: the slot list of this row (tables; no kernel writes them).  Launched as a programmatic
    // dependent, the CTA may be resident while the attention kernels still run; it reads partial results
    // only after the wait, and only then lets the kernel behind it (the next append) start, so that
    // kernel runs when the attention kernels have completed.
    unsigned int stamp = 0;
    if (a.stamps && threadIdx.x == 0) stamp = stamp_start(a.stamps, 3);
    MergeList ml{};
    if (active) ml = merge_list(a, (int)(row / a.Hq), (int)(row % a.Hq), lane);
    pdl_wait();
    pdl_launch_dependents();
    if (active) merge_row<D, kEarly>(a, (int)(row / a.Hq), (int)(row % a.Hq), lane, ml);
    if (a.stamps) {
        __syncthreads();
        if (threadIdx.x == 0) stamp_end(a.stamps, 3, stamp, gridDim.x);
    }
}

void launch_merge(const DecodeArgs& a, int D, bool chained, cudaStream_t s) {
    const int64_t rows = (int64_t)a.n_leaves * a.Hq;
    if (rows <= 0) return;
    const int blocks = (int)((rows + kMergeWarps - 1) / kMergeWarps);
    ChainLaunch l(dim3(blocks), dim3(kMergeWarps * 32), 0, s, chained);
    // A row usually has 8 to 12 partials.  With 12 of them fetched in the first round trip a warp needs more
    // registers and fewer CTAs fit on an SM: taken when the whole grid is resident at once even so (one
    // width-64 tree), where it saves the second round trip; larger grids keep 8 and the higher occupancy.
    const bool small_grid = blocks <= 148 * 4;
    if (D == 128) {
        if (small_grid) cudaLaunchKernelEx(&l.cfg, lse_merge_kernel<128, 12>, a);
        else cudaLaunchKernelEx(&l.cfg, lse_merge_kernel<128, 8>, a);
    } else {
        if (small_grid) cudaLaunchKernelEx(&l.cfg, lse_merge_kernel<64, 12>, a);
        else cudaLaunchKernelEx(&l.cfg, lse_merge_kernel<64, 8>, a);
    }
}

}  // namespace ets
