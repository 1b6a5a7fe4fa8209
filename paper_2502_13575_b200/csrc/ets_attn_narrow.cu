// Node-partial attention for narrow query groups (up to 16 query rows per work item).
//
// The work is HBM-bound: every (page, kv head) tile of K and V is read once and used for at most
// 16 query rows, i.e. at most 16 flop per byte.  The kernel is therefore organised around keeping
// bytes in flight, not around arithmetic:
//   * persistent grid, one CTA per SM, kNarrowWarps independent warps per CTA; a warp is a worker
//     with its own contiguous, cost-balanced piece of the work line, so no warp waits for another;
//   * every warp owns a ring of kDepth (2) shared-memory slots; a slot receives one K tile and one V
//     tile (16 tokens x D bf16 each) by two bulk asynchronous copies (TMA engine, linear form) that
//     complete on the slot's mbarrier; the ring runs ahead across item boundaries;
//   * a tile is stored in global memory as its shared-memory image (128-byte swizzle), so it lands
//     ready for ldmatrix without bank conflicts;
//   * the little arithmetic there is goes to the tensor cores in the "tokens as M" orientation:
//     S^T[16 tok x 8n rows] = K_tile . Q^T and O^T[D x 8n rows] += V_tile^T . P^T with
//     mma.sync.m16n8k16 (bf16 in, fp32 accumulate).  Padding the query rows to 8 costs nothing
//     here, and a scalar-FMA formulation cannot keep up with HBM beyond ~4 rows;
//   * online softmax in log2 units per 16-token tile; the partial (m, l, o) goes straight from
//     registers to global memory (a last-arriver merge fused in here was measured 3x slower than
//     the separate merge kernel: the merging warps stall their own streaming).
// Every wait on an mbarrier is bounded; on expiry the warp raises the status word, starts no new
// copy and only waits (again boundedly) for the few copies it had already started.
#include "ets_device.cuh"

namespace ets {

namespace {

constexpr int kWarps = kNarrowWarps;
constexpr int kDepth = 2;   // measured as fast as 3; 2 leaves shared memory for a wide-kernel CTA on the same SM
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// same copy with an L2 eviction-priority hint
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar), "l"(pol)
        : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void st_f32_hint(float* p, float v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(v), "l"(pol) : "memory");
}
__device__ __forceinline__ void st_f32x2_hint(float2* p, float2 v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.v2.f32 [%0], {%1, %2}, %3;" ::"l"(p), "f"(v.x), "f"(v.y), "l"(pol) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr)
                 : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr)
                 : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// A batch of up to 32 consecutive page slots of an item, one per lane: its page id and the number
// of tokens it holds now (0 = skip: empty, or a page id outside the pool, which is also flagged).
// Loading descriptors 32 at a time keeps the dependent global loads (slot -> node length) off the
// per-tile critical path.
struct UnitBatch {
    int base = 0;       // index (within the item) of lane 0's slot
    int page = 0;
    int valid = 0;
    uint32_t live = 0;  // bit i: lane i's slot has tokens

    __device__ __forceinline__ void load(const DecodeArgs& a, int unit_begin, int unit_count, int from, int lane) {
        base = from;
        const int idx = from + lane;
        page = 0;
        valid = 0;
        if (idx < unit_count) {
            const int4 un = a.units[unit_begin + idx];
            int v = a.node_len[un.y] - un.z;
            v = v < 0 ? 0 : (v > 16 ? 16 : v);
            if (v > 0 && (un.x < 0 || (int64_t)un.x >= a.pages_per_layer)) {  // never read outside the pool
                atomicExch(a.status, -1);
                v = 0;
            }
            page = un.x;
            valid = v;
        }
        live = __ballot_sync(0xffffffffu, valid > 0);
    }
    // first live slot at or after item index u inside this batch, or -1
    __device__ __forceinline__ int next_live(int u) const {
        const int sh = u - base;
        if (sh >= 32) return -1;
        const uint32_t m = live >> sh;
        return m ? u + __ffs(m) - 1 : -1;
    }
};

// Issue side of a warp's ring: walks the worker's items and their page slots, skipping slots that
// hold no token yet, and starts the two bulk copies of the next one.
template <int D>
struct Feeder {
    int it, it_end;       // next item index / end of this worker's items
    int u = 0, ub = 0, uc = 0, head = 0;
    bool reread = false;  // the current item's pages are read again by the next leaf tile
    uint64_t pol_stream;  // K/V read for the last time goes first when L2 needs room
    UnitBatch batch;
    uint32_t n_issued = 0;
    uint32_t ring, bars;  // shared-memory addresses of this warp's slots and barriers

    __device__ bool issue_next(const DecodeArgs& a, int lane) {
        constexpr uint32_t TB = 16 * D * 2;
        while (true) {
            if (u >= uc) {
                if (it >= it_end) return false;
                const DevItem d = a.items[it];
                ++it;
                ub = d.unit_begin; uc = d.unit_count; head = d.kv_head; u = 0;
                reread = (d.reserved & 1) != 0;
                batch.load(a, ub, uc, 0, lane);
                continue;
            }
            const int nxt = batch.next_live(u);
            if (nxt < 0) {
                u = batch.base + 32 < uc ? batch.base + 32 : uc;
                if (u < uc) batch.load(a, ub, uc, u, lane);
                continue;
            }
            const int page = __shfl_sync(0xffffffffu, batch.page, nxt - batch.base);
            u = nxt + 1;
            if (lane == 0) {
                const uint32_t slot = n_issued % kDepth;
                const uint32_t bar = bars + slot * 8;
                const uint32_t dst = ring + slot * 2 * TB;
                const size_t off = pool_tile_offset(a.pages_per_layer, page, head, TB);
                mbar_expect_tx(bar, 2 * TB);
                if (reread) {
                    bulk_g2s(dst, a.k_pool + off, TB, bar);
                    bulk_g2s(dst + TB, a.v_pool + off, TB, bar);
                } else {
                    bulk_g2s_hint(dst, a.k_pool + off, TB, bar, pol_stream);
                    bulk_g2s_hint(dst + TB, a.v_pool + off, TB, bar, pol_stream);
                }
            }
            ++n_issued;
            return true;
        }
    }
};

template <int D, int NT>
__device__ __forceinline__ void run_item(const DecodeArgs& a, const DevItem it, Feeder<D>& feed, uint32_t& n_consumed,
                                         bool& dead, int lane) {
    constexpr int KS = D / 16;
    constexpr uint32_t TB = 16 * D * 2;
    const int G = a.G;
    const int rows = it.n_leaves_tile * G;
    const int h = it.kv_head;
    const int quad = lane & 3, grp = lane >> 2;

    // Q^T fragments (B operand): row n = 8j + grp, features 16ks + 2quad + {0,1} and + 8
    uint32_t qf[NT][KS][2];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
        const int n = 8 * j + grp;
        if (n < rows) {
            const int leaf = a.node_leaves[it.leaf_list_begin + n / G];
            const uint32_t* qp = reinterpret_cast<const uint32_t*>(a.q + ((size_t)leaf * a.Hq + h * G + n % G) * D);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qf[j][ks][0] = qp[8 * ks + quad];
                qf[j][ks][1] = qp[8 * ks + 4 + quad];
            }
        } else {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) qf[j][ks][0] = qf[j][ks][1] = 0u;
        }
    }

    float o[KS][NT][4];
    float m[NT][2], l[NT][2];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
        m[j][0] = m[j][1] = -INFINITY;
        l[j][0] = l[j][1] = 0.f;
#pragma unroll
        for (int mt = 0; mt < KS; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[mt][j][i] = 0.f;
    }

    // per-lane pieces of the ldmatrix row addresses inside a tile
    const int mat = lane >> 3, r8 = lane & 7;
    const int k_tok = r8 + (mat & 1) * 8;    // K: matrices 0/1 = tokens 0-7 / 8-15, 2/3 = next 8 features
    const int k_cb = mat >> 1;
    const int v_tok = r8 + (mat >> 1) * 8;   // V^T: matrices 0/1 = features +0 / +8, 2/3 = tokens 8-15
    const int v_cb = mat & 1;
    const uint32_t k_row = (uint32_t)(k_tok >> 3) * (D / 64) * 1024u + (uint32_t)(k_tok & 7) * 128u;
    const uint32_t v_row = (uint32_t)(v_tok >> 3) * (D / 64) * 1024u + (uint32_t)(v_tok & 7) * 128u;

    UnitBatch cb;
    cb.load(a, it.unit_begin, it.unit_count, 0, lane);
    for (int u = 0; u < it.unit_count;) {
        const int nxt = cb.next_live(u);
        if (nxt < 0) {
            u = cb.base + 32 < it.unit_count ? cb.base + 32 : it.unit_count;
            if (u < it.unit_count) cb.load(a, it.unit_begin, it.unit_count, u, lane);
            continue;
        }
        const int valid = __shfl_sync(0xffffffffu, cb.valid, nxt - cb.base);
        u = nxt + 1;
        const uint32_t slot = n_consumed % kDepth;
        const uint32_t parity = (n_consumed / kDepth) & 1u;
        const bool issued = n_consumed < feed.n_issued;
        ++n_consumed;
        if (dead) {
            // gave up earlier: only wait (boundedly) for copies already started, so that none
            // lands after the CTA has gone; nothing new is issued
            if (issued) mbar_wait_bounded(feed.bars + slot * 8, parity);
            continue;
        }
        if (!mbar_wait_bounded(feed.bars + slot * 8, parity)) {
            if (lane == 0) atomicExch(a.status, -7);
            dead = true;
            continue;
        }
        const uint32_t kt = feed.ring + slot * 2 * TB;
        const uint32_t vt = kt + TB;

        if (valid < 16) {
            // rows past the node's length hold stale bytes: zero them in V so that 0 * garbage
            // cannot produce NaN (their scores are masked below)
            for (int i = lane; i < (16 - valid) * (D / 8); i += 32) {
                const int t = valid + i / (D / 8), c = i % (D / 8);
                asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + tile_offset(D, t, c * 8)), "r"(0u) : "memory");
            }
            __syncwarp();
        }

        // S^T = K_tile . Q^T
        float s[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int chunk = 2 * ks + k_cb;
            uint32_t af[4];
            ldsm_x4(kt + k_row + (uint32_t)(chunk >> 3) * 1024u + (uint32_t)(((chunk & 7) ^ (k_tok & 7)) << 4), af);
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_bf16(s[j], af, qf[j][ks]);
        }

        // online softmax (log2 units); this lane holds tokens grp and grp+8 of rows 2quad, 2quad+1
        uint32_t pf[NT][2];
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            float sv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int tok = grp + (i >> 1) * 8;
                sv[i] = tok < valid ? s[j][i] * a.scale_log2 : -INFINITY;
            }
            float p[4];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                float mx = fmaxf(sv[r], sv[r + 2]);
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                const float mn = fmaxf(m[j][r], mx);     // finite: token 0 of the tile is valid
                const float corr = exp2f(m[j][r] - mn);
                // weights are rounded to bf16 here, so that the row sum and the product use the same
                // values and the rounding cancels in sum(p v) / sum(p)
                p[r] = __bfloat162float(__float2bfloat16_rn(exp2f(sv[r] - mn)));
                p[r + 2] = __bfloat162float(__float2bfloat16_rn(exp2f(sv[r + 2] - mn)));
                l[j][r] = l[j][r] * corr + p[r] + p[r + 2];
                m[j][r] = mn;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    o[mt][j][r] *= corr;
                    o[mt][j][r + 2] *= corr;
                }
            }
            // P^T as B operand: transpose the two 8x8 (token x row) blocks
            pf[j][0] = movmatrix_trans(pack_bf16(p[0], p[1]));
            pf[j][1] = movmatrix_trans(pack_bf16(p[2], p[3]));
        }

        // O^T += V_tile^T . P^T
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
            const int chunk = 2 * mt + v_cb;
            uint32_t af[4];
            ldsm_x4_trans(vt + v_row + (uint32_t)(chunk >> 3) * 1024u + (uint32_t)(((chunk & 7) ^ (v_tok & 7)) << 4), af);
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_bf16(o[mt][j], af, pf[j]);
        }

        // the slot is free again: order our shared-memory reads (and the zero fill) before the
        // next asynchronous write into it, then refill
        __syncwarp();
        fence_proxy_async();
        feed.issue_next(a, lane);
    }

    // partial (m, l, o) of this item, straight from registers
    const uint64_t pol_keep = policy_evict_last();
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float ls = l[j][r];
            ls += __shfl_xor_sync(0xffffffffu, ls, 4);
            ls += __shfl_xor_sync(0xffffffffu, ls, 8);
            ls += __shfl_xor_sync(0xffffffffu, ls, 16);
            const int n = 8 * j + 2 * quad + r;
            if (n < rows) {
                const size_t prow = (size_t)(it.slot_first + n / G) * G + n % G;
                // partials are read back by the merge kernel right after: ask L2 to hold on to them
                if (grp == 0) st_f32x2_hint(a.part_ml + prow, make_float2(m[j][r], ls), pol_keep);
                float* po = a.part_o + prow * D + grp;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    st_f32_hint(po + 16 * mt, o[mt][j][r], pol_keep);
                    st_f32_hint(po + 16 * mt + 8, o[mt][j][r + 2], pol_keep);
                }
            }
        }
}

template <int D>
// 168 registers x 256 threads leave room in the register file for a wide-kernel CTA (96 x 192)
__global__ void __maxnreg__(168) attn_partial_narrow_kernel(DecodeArgs a) {
    constexpr uint32_t TB = 16 * D * 2;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (base & 127u) {   // the swizzled tile rows must start on 128-byte boundaries
        if (threadIdx.x == 0) atomicExch(a.status, -1);
        return;
    }

    const int worker = blockIdx.x * kWarps + warp;
    if (worker >= a.n_workers) return;
    const int i0 = a.worker_off[worker], i1 = a.worker_off[worker + 1];
    if (i0 >= i1) return;

    Feeder<D> feed;
    feed.it = i0;
    feed.it_end = i1;
    feed.pol_stream = policy_evict_first();
    feed.ring = base + (uint32_t)warp * kDepth * 2 * TB;
    feed.bars = base + (uint32_t)kWarps * kDepth * 2 * TB + (uint32_t)warp * kDepth * 8;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kDepth; ++s) mbar_init(feed.bars + s * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

#pragma unroll
    for (int s = 0; s < kDepth; ++s) feed.issue_next(a, lane);

    uint32_t n_consumed = 0;
    bool dead = false;
    for (int i = i0; i < i1; ++i) {
        const DevItem it = a.items[i];
        if (it.n_leaves_tile * a.G <= 8) run_item<D, 1>(a, it, feed, n_consumed, dead, lane);
        else run_item<D, 2>(a, it, feed, n_consumed, dead, lane);
    }
}

}  // namespace

size_t narrow_smem_bytes(int D) { return (size_t)kWarps * kDepth * 2 * 16 * D * 2 + kWarps * kDepth * 8; }

cudaError_t narrow_prepare(int D) {
    // the largest shared-memory carve-out, so that a CTA of the other attention kernel can be
    // resident on the same SM
    cudaError_t e;
    if (D == 128) {
        e = cudaFuncSetAttribute(attn_partial_narrow_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)narrow_smem_bytes(128));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_partial_narrow_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    } else {
        e = cudaFuncSetAttribute(attn_partial_narrow_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)narrow_smem_bytes(64));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_partial_narrow_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    }
    return e;
}

void launch_partial_narrow(const DecodeArgs& a, int D, int n_ctas, cudaStream_t s) {
    if (a.n_items <= 0 || n_ctas <= 0) return;
    if (D == 128) attn_partial_narrow_kernel<128><<<n_ctas, kWarps * 32, narrow_smem_bytes(128), s>>>(a);
    else attn_partial_narrow_kernel<64><<<n_ctas, kWarps * 32, narrow_smem_bytes(64), s>>>(a);
}

}  // namespace ets
