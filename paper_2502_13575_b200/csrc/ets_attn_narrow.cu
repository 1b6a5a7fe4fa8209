// Node-partial attention for narrow query groups (up to 16 query rows per work item).
//
// The work is HBM-bound: every (page, kv head) tile of K and V is read once and used for at most
// 16 query rows, i.e. at most 16 flop per byte.  The kernel is therefore organised around keeping
// bytes in flight, not around arithmetic:
//   * persistent grid, one CTA per SM, kNarrowWarps independent warps per CTA; a warp is a worker
//     that takes work items from a queue ordered longest first: item w for warp w, then whatever
//     a shared counter hands out, so a warp that is early simply takes more; the next item
//     (descriptor, page slots, lengths) is fetched in the background, one dependent load per tile;
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
#include <climits>

#include "ets_device.cuh"

namespace ets {

namespace {

constexpr int kWarps = kNarrowWarps;
#ifndef ETS_DEPTH
#define ETS_DEPTH 2
#endif
constexpr int kDepth = ETS_DEPTH;   // measured as fast as 3; 2 leaves shared memory for a wide-kernel CTA on the same SM
constexpr uint32_t kSpinLimit = kWaitPolls;
#ifndef ETS_CLAIM_AHEAD
#define ETS_CLAIM_AHEAD 6
#endif
constexpr int kClaimAhead = ETS_CLAIM_AHEAD;   // tiles left in the current item when the next one is claimed

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
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t polls = kSpinLimit) {
    for (uint32_t i = 0; i < polls; ++i)
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
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The page slots of one narrow item, one per lane (an item has at most 32): where the page's tiles are and the number
// of tokens the slot holds now (0 = skip: empty, or a page id outside the pool, which is also flagged).
struct SlotView {
    int page = 0;       // bit 0: which pool buffer holds the page; bits 1..: index of its (K tile, V tile) pair there, for the item's kv head
    int valid = 0;
    uint32_t live = 0;  // bit i: lane i's slot has tokens
};

// The next item of this warp, fetched in the background while the current one is processed.  The
// chain claim -> descriptor -> page slots -> node lengths is four dependent memory round trips;
// one link is started per consumed tile, so that none of them stalls the warp.
struct NextItem {
    int stage = 4;      // 0 nothing claimed, 1 claim in flight, 2 descriptor in flight, 3 slots in flight, 4 complete
    int idx = INT_MAX;  // queue position; >= n_narrow: the queue is empty
    int claim = 0;      // lane 0: value returned by the shared counter
    DevItem it{};
    int4 un = make_int4(0, 0, 0, 0);
    int leaf[2] = {0, 0};   // leaf of query rows grp and 8 + grp
    SlotView v;
};

template <int D, int NT>
struct Acc {
    float o[D / 16][NT][4];
    float m[NT][2], l[NT][2];
};

// Q^T fragments (B operand) of an item: row n = 8j + grp, features 16ks + 2quad + {0,1} and + 8
template <int D, int NT>
__device__ __forceinline__ void load_q(const DecodeArgs& a, const DevItem& it, const int (&leaf)[2], int lane,
                                       uint32_t (&qf)[NT][D / 16][2]) {
    constexpr int KS = D / 16;
    const int G = a.G, rows = it.n_leaves_tile * G, quad = lane & 3, grp = lane >> 2;
#pragma unroll
    for (int j = 0; j < NT; ++j) {
        const int n = 8 * j + grp;
        if (n < rows) {
            const uint32_t* qp = reinterpret_cast<const uint32_t*>(a.q + ((size_t)leaf[j] * a.Hq + it.kv_head * G + n % G) * D);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qf[j][ks][0] = __ldg(qp + 8 * ks + quad);
                qf[j][ks][1] = __ldg(qp + 8 * ks + 4 + quad);
            }
        } else {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) qf[j][ks][0] = qf[j][ks][1] = 0u;
        }
    }
}

// One K tile and one V tile (16 tokens) against the item's query rows: S^T = K . Q^T, online softmax
// in log2 units, O^T += V^T . P^T.
template <int D, int NT>
__device__ __forceinline__ void tile_step(uint32_t kt, uint32_t vt, int valid, float scale_log2, int lane,
                                          const uint32_t (&qf)[NT][D / 16][2], Acc<D, NT>& acc) {
    constexpr int KS = D / 16;
    const int grp = lane >> 2;
    // per-lane pieces of the ldmatrix row addresses inside a tile
    const int mat = lane >> 3, r8 = lane & 7;
    const int k_tok = r8 + (mat & 1) * 8;    // K: matrices 0/1 = tokens 0-7 / 8-15, 2/3 = next 8 features
    const int v_tok = r8 + (mat >> 1) * 8;   // V^T: matrices 0/1 = features +0 / +8, 2/3 = tokens 8-15
    // chunk index 2*ks + cb, XOR-swizzled by the row: (2ks | cb) ^ r8 = (2ks) ^ (cb ^ r8)
    const uint32_t k_lane = kt + (uint32_t)(k_tok >> 3) * (D / 64) * 1024u + (uint32_t)r8 * 128u + (uint32_t)(((mat >> 1) ^ r8) << 4);
    const uint32_t v_lane = vt + (uint32_t)(v_tok >> 3) * (D / 64) * 1024u + (uint32_t)r8 * 128u + (uint32_t)(((mat & 1) ^ r8) << 4);

    if (valid < 16) {
        // rows past the node's length hold stale bytes: zero them in V so that 0 * garbage
        // cannot produce NaN (their scores are masked below)
        for (int i = lane; i < (16 - valid) * (D / 8); i += 32) {
            const int t = valid + i / (D / 8), c = i % (D / 8);
            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + tile_offset(D, t, c * 8)), "r"(0u) : "memory");
        }
        __syncwarp();
    }

    // S^T = K_tile . Q^T; with a single column tile the k-steps alternate between two accumulators, so
    // that the chain of dependent products is half as long
    constexpr int NS = NT == 1 ? 2 : 1;
    float s[NT][4], s2[NS][4];
#pragma unroll
    for (int j = 0; j < NT; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
    s2[0][0] = s2[0][1] = s2[0][2] = s2[0][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        uint32_t af[4];
        ldsm_x4((k_lane + (uint32_t)(ks >> 2) * 1024u) ^ (uint32_t)((ks & 3) << 5), af);
        if (NT == 1 && (ks & 1)) {
            mma_bf16(s2[0], af, qf[0][ks]);
        } else {
#pragma unroll
            for (int j = 0; j < NT; ++j) mma_bf16(s[j], af, qf[j][ks]);
        }
    }
    if (NT == 1) {
#pragma unroll
        for (int i = 0; i < 4; ++i) s[0][i] += s2[0][i];
    }

    // online softmax (log2 units); this lane holds tokens grp and grp+8 of rows 2quad, 2quad+1.  The two rows
    // go through the packed fp32 instructions together (one instruction for both): the warp is a chain of
    // dependent instructions and their number is what a tile costs.
    uint32_t pf[NT][2], pg[NT][2];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
        const float2 sc2 = make_float2(scale_log2, scale_log2);
        // (row 2quad, row 2quad+1) of token grp and of token grp+8; tokens past the node's length are masked
        float2 sa = __fmul2_rn(make_float2(s[j][0], s[j][1]), sc2);
        float2 sb = __fmul2_rn(make_float2(s[j][2], s[j][3]), sc2);
        if (grp >= valid) sa = make_float2(-INFINITY, -INFINITY);
        if (grp + 8 >= valid) sb = make_float2(-INFINITY, -INFINITY);
        float2 mx = make_float2(fmaxf(sa.x, sb.x), fmaxf(sa.y, sb.y));
#pragma unroll
        for (int d = 4; d <= 16; d <<= 1) {
            mx.x = fmaxf(mx.x, __shfl_xor_sync(0xffffffffu, mx.x, d));
            mx.y = fmaxf(mx.y, __shfl_xor_sync(0xffffffffu, mx.y, d));
        }
        // finite: token 0 of the tile is valid
        const float2 mn = make_float2(fmaxf(acc.m[j][0], mx.x), fmaxf(acc.m[j][1], mx.y));
        const float2 neg = make_float2(-mn.x, -mn.y);
        const float2 corr = make_float2(ex2_approx(acc.m[j][0] + neg.x), ex2_approx(acc.m[j][1] + neg.y));
        const float2 da = __fadd2_rn(sa, neg), db = __fadd2_rn(sb, neg);
        // weights are at most 1 and are rounded to bf16 next: the approximate exponential (2 ulp, tiny results
        // flushed to zero) loses nothing
        const float2 ea = make_float2(ex2_approx(da.x), ex2_approx(da.y));
        const float2 eb = make_float2(ex2_approx(db.x), ex2_approx(db.y));
        // A weight enters the product as two bf16 terms, its rounded value and the rounded rest
        // (16 bits of it in all): with one term the weights would be off by up to 2^-8 each, which
        // on a path of a few tokens with values of opposite sign exceeds the output's tolerance.
        const __nv_bfloat162 pa = __floats2bfloat162_rn(ea.x, ea.y);
        const __nv_bfloat162 pb = __floats2bfloat162_rn(eb.x, eb.y);
        const float2 minus1 = make_float2(-1.f, -1.f);
        const float2 ra = __ffma2_rn(make_float2(__low2float(pa), __high2float(pa)), minus1, ea);
        const float2 rb = __ffma2_rn(make_float2(__low2float(pb), __high2float(pb)), minus1, eb);
        const __nv_bfloat162 qa = __floats2bfloat162_rn(ra.x, ra.y);
        const __nv_bfloat162 qb = __floats2bfloat162_rn(rb.x, rb.y);
        const float2 l2 = __fadd2_rn(__ffma2_rn(make_float2(acc.l[j][0], acc.l[j][1]), corr, ea), eb);
        acc.l[j][0] = l2.x;
        acc.l[j][1] = l2.y;
        acc.m[j][0] = mn.x;
        acc.m[j][1] = mn.y;
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
            const float2 o01 = __fmul2_rn(make_float2(acc.o[mt][j][0], acc.o[mt][j][1]), corr);
            const float2 o23 = __fmul2_rn(make_float2(acc.o[mt][j][2], acc.o[mt][j][3]), corr);
            acc.o[mt][j][0] = o01.x;
            acc.o[mt][j][1] = o01.y;
            acc.o[mt][j][2] = o23.x;
            acc.o[mt][j][3] = o23.y;
        }
        // P^T as B operand: transpose the two 8x8 (token x row) blocks
        pf[j][0] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&pa));
        pf[j][1] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&pb));
        pg[j][0] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&qa));
        pg[j][1] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&qb));
    }

    // O^T += V_tile^T . P^T
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) {
        uint32_t af[4];
        ldsm_x4_trans((v_lane + (uint32_t)(mt >> 2) * 1024u) ^ (uint32_t)((mt & 3) << 5), af);
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_bf16(acc.o[mt][j], af, pf[j]);
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_bf16(acc.o[mt][j], af, pg[j]);
    }
}

// partial (m, l, o) of an item, straight from registers
template <int D, int NT>
__device__ __forceinline__ void store_partials(const DecodeArgs& a, const DevItem& it, int lane, Acc<D, NT>& acc) {
    constexpr int KS = D / 16;
    const int G = a.G, rows = it.n_leaves_tile * G, quad = lane & 3, grp = lane >> 2;
    const uint64_t pol_keep = policy_evict_last();
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float ls = acc.l[j][r];
            ls += __shfl_xor_sync(0xffffffffu, ls, 4);
            ls += __shfl_xor_sync(0xffffffffu, ls, 8);
            ls += __shfl_xor_sync(0xffffffffu, ls, 16);
            const int n = 8 * j + 2 * quad + r;
            if (n < rows) {
                // rows of an item are consecutive: (slot_first + n / G) * G + n % G = slot_first * G + n
                const size_t prow = (size_t)it.slot_first * G + n;
                // partials are read back by the merge kernel right after: ask L2 to hold on to them
                if (grp == 0) st_f32x2_hint(a.part_ml + prow, make_float2(acc.m[j][r], ls), pol_keep);
                float* po = a.part_o + prow * D + grp;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    st_f32_hint(po + 16 * mt, acc.o[mt][j][r], pol_keep);
                    st_f32_hint(po + 16 * mt + 8, acc.o[mt][j][r + 2], pol_keep);
                }
            }
        }
}

template <int N>
struct IntTag { static constexpr int value = N; };

// Device time stamps of the narrow kernel, out of line so that they do not weigh on the register allocation of the
// streaming loop: what = 0 at kernel entry, 1 when the wait for the kernel ahead has returned, 2 when a warp is done.
__device__ __noinline__ void narrow_stamp(Stamps* s, int what, int n_warps) {
    if (what == 0) {
        if (threadIdx.x == 0) stamp_start(s, 1);
    } else if (what == 1) {
        if (threadIdx.x == 0) stamp_start(s, 4);
    } else if ((threadIdx.x & 31) == 0) {
        // no warp of this launch has finished yet when any of them reads the index, so all read the same one
        const unsigned int i = min(*((volatile unsigned int*)&s->count[1]), (unsigned int)kStampLaunches);
        if (threadIdx.x == 0 && blockIdx.x == 0) stamp_end(s, 4, i, 1);   // the "wait returned" series advances with the launch
        stamp_end(s, 1, i, (unsigned int)n_warps);
    }
}

template <int D>
// 168 registers x 256 threads leave room in the register file for a wide-kernel CTA (80 x 192)
__global__ void __maxnreg__(168) attn_partial_narrow_kernel(DecodeArgs a) {
    constexpr uint32_t TB = 16 * D * 2;
    constexpr uint32_t FULL = 0xffffffffu;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_warps = (int)gridDim.x * kWarps;
    const int worker = blockIdx.x * kWarps + warp;
    const int grp = lane >> 2;
    const int G = a.G;

    if (a.stamps) narrow_stamp(a.stamps, 0, 0);
    const bool aligned = (base & 127u) == 0;   // the swizzled tile rows must start on 128-byte boundaries
    const bool active = aligned && worker < a.n_narrow;
    if (!aligned && threadIdx.x == 0) atomicExch(a.status, -1);
    {
        const uint32_t ring = base + (uint32_t)warp * kDepth * 2 * TB;
        const uint32_t bars = base + (uint32_t)kWarps * kDepth * 2 * TB + (uint32_t)warp * kDepth * 8;
        if (active && lane == 0) {
#pragma unroll
            for (int s = 0; s < kDepth; ++s) mbar_init(bars + s * 8, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        const uint64_t pol_stream = policy_evict_first();   // K/V read for the last time goes first when L2 needs room

        uint32_t n_issued = 0, n_consumed = 0;
        DevItem cur{};
        SlotView cv;
        int cur_leaf[2] = {0, 0};
        bool f_on_next = false;     // the issue side has moved on to the next item
        uint32_t f_live = 0;        // slots of its item that it has not started yet
        int f_page = 0;             // its item: per lane, where the slot's tile pair sits (see SlotView::page)
        bool f_reread = false;      // its item's pages are read again by the next leaf tile
        NextItem nx;

        // one link of the background fetch of the next item
        auto fetch_step = [&]() {
            switch (nx.stage) {
                case 0:
                    if (lane == 0) nx.claim = atomicAdd(a.queue, 1);
                    nx.stage = 1;
                    break;
                case 1:
                    nx.idx = n_warps + __shfl_sync(FULL, nx.claim, 0);
                    if (nx.idx < a.n_narrow) {
                        nx.it = a.items[nx.idx];
                        nx.stage = 2;
                    } else {
                        nx.idx = INT_MAX;
                        nx.stage = 4;
                    }
                    break;
                case 2: {
                    nx.un = lane < nx.it.unit_count ? a.units[nx.it.unit_begin + lane] : make_int4(0, 0, 0, 0);
                    const int rows = nx.it.n_leaves_tile * G;
#pragma unroll
                    for (int j = 0; j < 2; ++j)
                        nx.leaf[j] = 8 * j + grp < rows ? a.node_leaves[nx.it.leaf_list_begin + (8 * j + grp) / G] : 0;
                    nx.stage = 3;
                    break;
                }
                case 3: {
                    int v = 0;
                    if (lane < nx.it.unit_count) {
                        v = a.node_len[nx.un.y] - nx.un.z;
                        v = v < 0 ? 0 : (v > 16 ? 16 : v);
                        if (v > 0 && (nx.un.x < 0 || (int64_t)nx.un.x >= a.pages_per_layer)) {  // never read outside the pool
                            atomicExch(a.status, -1);
                            v = 0;
                        }
                    }
                    // tile pair index inside its pool buffer, and which buffer (see kv_tile), worked out here by all
                    // lanes at once instead of by the one lane that later starts the copy
                    nx.v.page = (int)((((uint32_t)nx.it.kv_head * (uint32_t)pool_pairs(a.pages_per_layer) + (uint32_t)(nx.un.x >> 1)) << 1) | (uint32_t)(nx.un.x & 1));
                    nx.v.valid = v;
                    nx.v.live = __ballot_sync(FULL, v > 0);
                    nx.stage = 4;
                    break;
                }
                default:
                    break;
            }
        };
        auto fetch_finish = [&]() {
            while (nx.stage < 4) fetch_step();
        };

        // Issue side of the ring: starts the two bulk copies of the next page slot that holds tokens,
        // in the current item or, once that is exhausted, in the next one.
        auto issue_next = [&]() -> bool {
            while (true) {
                if (f_live) {
                    const int b = __ffs(f_live) - 1;
                    f_live &= f_live - 1;
                    const uint32_t where = (uint32_t)__shfl_sync(FULL, f_page, b);
                    if (lane == 0) {
                        const uint32_t slot = n_issued % kDepth;
                        const uint32_t bar = bars + slot * 8;
                        const uint32_t dst = ring + slot * 2 * TB;
                        const char* src = ((where & 1u) ? a.v_pool : a.k_pool) + (size_t)(where >> 1) * (2 * TB);
                        mbar_expect_tx(bar, 2 * TB);
                        if (f_reread) bulk_g2s(dst, src, 2 * TB, bar);   // K tile and V tile in one copy
                        else bulk_g2s_hint(dst, src, 2 * TB, bar, pol_stream);
                    }
                    ++n_issued;
                    return true;
                }
                if (f_on_next) return false;   // nothing is known beyond the next item yet
                fetch_finish();
                if (nx.idx == INT_MAX) return false;   // the queue is empty
                // the issue side keeps its own copy of what it needs of its item, so that it never
                // touches the registers of a fetch that is still in flight
                f_on_next = true;
                f_live = nx.v.live;
                f_page = nx.v.page;
                f_reread = (nx.it.reserved & 1) != 0;
            }
        };

        // The first item of this warp is its own index in the queue.  Its descriptor, page slots and leaf
        // ids come from the tables, which no kernel writes: they are fetched before the wait for the
        // kernel ahead in the stream (launched as its programmatic dependent, this part runs under that
        // kernel's tail).  Node lengths, K/V, the queue counter and the partial results are touched
        // only after the wait; only then may the kernel behind this one (the wide-group kernel) start,
        // so that its start implies that the appended K/V and lengths are complete.
        if (active) {
            nx.idx = worker;
            nx.it = a.items[worker];
            nx.stage = 2;
            fetch_step();
        } else {
            nx.idx = INT_MAX;
        }
        pdl_wait();
        pdl_launch_dependents();
        if (a.stamps) narrow_stamp(a.stamps, 1, 0);
        if (active) fetch_finish();

        bool dead = false;
        bool first_wait = true;
        while (nx.idx != INT_MAX && !dead) {
            // make the fetched item the current one and start fetching its successor
            cur = nx.it;
            cv = nx.v;
            cur_leaf[0] = nx.leaf[0];
            cur_leaf[1] = nx.leaf[1];
            if (f_on_next) {
                f_on_next = false;
            } else {
                f_live = cv.live;
                f_page = cv.page;
                f_reread = (cur.reserved & 1) != 0;
            }
            nx.stage = 0;
            nx.idx = INT_MAX;
            if (__popc(cv.live) <= kClaimAhead) fetch_step();
            while (n_issued - n_consumed < (uint32_t)kDepth && issue_next()) {}

            auto process = [&](auto tag) {
                constexpr int NT = decltype(tag)::value;
                constexpr int KS = D / 16;
                uint32_t qf[NT][KS][2];
                load_q<D, NT>(a, cur, cur_leaf, lane, qf);
                Acc<D, NT> acc;
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    acc.m[j][0] = acc.m[j][1] = -INFINITY;
                    acc.l[j][0] = acc.l[j][1] = 0.f;
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc.o[mt][j][i] = 0.f;
                }
                uint32_t todo = cv.live;
                while (todo) {
                    const int b = __ffs(todo) - 1;
                    todo &= todo - 1;
                    const int valid = __shfl_sync(FULL, cv.valid, b);
                    const uint32_t slot = n_consumed % kDepth;
                    const uint32_t parity = (n_consumed / kDepth) & 1u;
                    ++n_consumed;
                    const uint32_t polls = first_wait ? a.first_wait_polls : kSpinLimit;
                    first_wait = false;
                    if (!__all_sync(FULL, mbar_wait_bounded(bars + slot * 8, parity, polls))) {   // same answer in every lane
                        if (lane == 0) atomicExch(a.status, -7);
                        dead = true;
                        return;
                    }
                    const uint32_t kt = ring + slot * 2 * TB;
                    tile_step<D, NT>(kt, kt + TB, valid, a.scale_log2, lane, qf, acc);
                    // The slot is free again once every lane has its fragments (their values have been
                    // consumed by the products above).  Only the zero fill of a partial page is a write
                    // through the generic proxy that the next asynchronous copy must be ordered after.
                    __syncwarp();
                    if (valid < 16) fence_proxy_async();
                    issue_next();
                    // the successor is claimed late (an early claim would tie work to this warp while
                    // others run out of it), but early enough for its four loads to finish in time
                    if (__popc(todo) < kClaimAhead) fetch_step();
                }
                store_partials<D, NT>(a, cur, lane, acc);
            };
            if (cur.n_leaves_tile * G <= 8) process(IntTag<1>{});
            else process(IntTag<2>{});
            if (!dead) fetch_finish();
        }
        if (dead) {
            // gave up: nothing new is started; wait (boundedly) for the copies already started, so that
            // none lands after the CTA has gone.  The slot whose wait ran out counts as consumed.  A claim
            // on the item queue that is still in flight is waited for too (by using its value), so that it
            // cannot land after the last warp has rewound the counter.
            if (nx.stage == 1 && __shfl_sync(FULL, nx.claim, 0) < 0) atomicExch(a.status, -1);
            while (n_consumed < n_issued) {
                mbar_wait_bounded(bars + (n_consumed % kDepth) * 8, (n_consumed / kDepth) & 1u);
                ++n_consumed;
            }
        }
    }

    // Every warp of the grid reports here; the last one rewinds the queue for the next launch.  A warp's
    // claims have all returned before it gets here, so nobody touches the counter after the last report.
    __syncwarp();
    if (a.stamps) narrow_stamp(a.stamps, 2, n_warps);
    if (lane == 0 && atomicAdd(a.queue + 1, 1) == n_warps - 1) {
        a.queue[0] = 0;
        a.queue[1] = 0;
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

void launch_partial_narrow(const DecodeArgs& a, int D, int n_ctas, bool chained, cudaStream_t s) {
    if (a.n_narrow <= 0 || n_ctas <= 0) return;
    ChainLaunch l(dim3(n_ctas), dim3(kWarps * 32), narrow_smem_bytes(D), s, chained);
    if (D == 128) cudaLaunchKernelEx(&l.cfg, attn_partial_narrow_kernel<128>, a);
    else cudaLaunchKernelEx(&l.cfg, attn_partial_narrow_kernel<64>, a);
}

}  // namespace ets
