// Node-partial attention for wide query groups (17 .. 128 query rows per work item) on the
// 5th-generation tensor cores: tcgen05.mma with accumulators in tensor memory.
//
// A wide group is where the path really is a dense contraction: one K/V tile serves up to 128
// query rows, so both products are issued as UMMA instructions with M = 128 (query rows, one per
// TMEM lane) instead of being re-read once per 16 rows by the narrow kernel.
//
// One CTA per work item, six warps:
//   warp 0      producer: walks the item's page slots, skips empty ones, and brings up to four
//               K tiles and four V tiles (64 tokens) per stage into shared memory with linear
//               bulk copies; the page image in global memory already is the SWIZZLE_128B operand
//               layout, so no tensor map is needed.  Also owns the TMEM allocation.
//   warp 1      MMA issuer: S = Q . K^T   (A = Q from shared memory, K-major; B = K stage, K-major)
//               then       O += P . V     (A = P from tensor memory;  B = V stage, MN-major).
//   warps 2-5   softmax: one query row per thread (its TMEM lane); scores in log2 units, online
//               maximum; when a row's maximum grows, O is rescaled in tensor memory.  (Raising the
//               reference lazily, only after it is outgrown by 2^8, saves most rescales but leaves
//               the dominant weight off a power of two, and its bf16 rounding then shows in peaked
//               rows whose output nearly cancels; the exact policy keeps that weight at 1.)
// A CTA holds two stages of 64 tokens and two S buffers in tensor memory.  The K half and the V half of a
// stage are tracked separately: a K half is free again as soon as its S = Q K^T has run, one whole stage
// before the V half (free after O += P V), so K of stage s + 2 is already on its way while the softmax warps
// work on stage s, and S of stage s + 1 is in tensor memory before they are done.  The tensor pipe runs
// QK(0) QK(1) PV(0) QK(2) PV(1) QK(3) ...: a product never waits for a copy that was started less than a
// stage ago, and what is left on the critical path of a stage is the softmax itself (maximum pass, rescale of
// O, exponentials) plus the hand-over to PV.  A CTA alone does not saturate anything; it is sized (97 KB of
// shared memory, 256 TMEM columns) to sit on an SM next to a CTA of the narrow kernel, launched behind it as
// its programmatic dependent, and the two overlap.
// Every wait is bounded.  A wait that runs out sets an abort flag that all roles poll, the status
// word is raised, copies in flight are waited for (again boundedly), TMEM is released, and the CTA
// returns.
#include "ets_device.cuh"

namespace ets {

namespace {

constexpr int kWideThreads = 192;
constexpr int kStageUnits = 4;                 // page slots (16 tokens each) per stage
constexpr int kStages = 2;                     // two 64-token stages in shared memory (K half and V half each)
constexpr int kInfoRing = 4;                   // stage descriptions outlive the K half they were written with (see Shared)
constexpr uint32_t kSpin = kWaitPolls;
constexpr uint32_t kTmemCols = 256;
// P (bf16, 8 columns per 16 tokens) is written over the S columns it was computed from: chunk c of P
// covers columns that only hold S chunks <= c/2, which the thread has consumed by then.
// S has two buffers of 64 columns (a stage is 64 tokens): the product of the next stage is issued while the
// softmax warps still work on this one.
constexpr uint32_t kColS = 0, kColP = 0, kColO = 128, kColSBuf = 64;
// P of a pair of page slots replaces the pair's S (32 columns): 16 columns of bf16 weights, then 16 columns
// with their second bf16 term (what rounding the first left over)
constexpr uint32_t kColPLo = 16;
__host__ __device__ constexpr uint32_t p_col(int k) { return 32u * (uint32_t)(k >> 1) + 8u * (uint32_t)(k & 1); }
static_assert(kStageUnits * 16 <= (int)kColSBuf && kStages == 2, "S double buffer: 64-token stages, two of them");
constexpr float kRescaleThreshold = 0.0f;      // log2 units; see the softmax role

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: SWIZZLE_128B, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, M = 128, N given, B either K- or MN-major.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)acc)
        : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
        "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
        "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// maximum of three (one instruction on sm_100)
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

struct StageInfo {
    int32_t n_units;                 // page slots in the stage (0 = end of item)
    int32_t page[kStageUnits];       // page of each (the V copies are started later than the K copies)
    int32_t valid[kStageUnits];      // tokens held by each
    int32_t node[kStageUnits];       // node it belongs to and index of its first token there: a query that
    int32_t tok0[kStageUnits];       // is limited inside its own node (step prefill) needs them
};

struct Shared {
    uint64_t full_k[kStages];        // K copies of a stage have landed (producer -> MMA warp)
    uint64_t full_v[kStages];        // V copies of a stage have landed
    uint64_t empty_k[kStages];       // K half may be overwritten (QK product done -> producer)
    uint64_t empty_v[kStages];       // V half may be overwritten (PV product done -> producer)
    uint64_t s_ready[2];             // S = Q K^T of an even / odd stage is in tensor memory (MMA -> softmax)
    uint64_t p_ready;                // P is in tensor memory (softmax -> MMA), 4 arrivals
    uint64_t o_ready;                // O += P V done (MMA -> softmax)
    uint32_t tmem_base;
    volatile int32_t abort;
    // Stage st is described in info[st % 4]: it is written when the K copies of st start (QK(st - 2) done,
    // which is before the softmax of st - 2 has read its own description) and read until PV(st) is issued;
    // entry st % 4 is next written for st + 4, after QK(st + 2), which the tensor pipe runs after PV(st).
    StageInfo info[kInfoRing];
};

// Called by all 32 lanes of a warp together; the answer is the same in every lane, so that the
// warp-collective tcgen05 instructions that follow are never reached by only part of a warp.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, Shared* sh, uint32_t polls = kSpin) {
    bool ok = false;
    for (uint32_t i = 0; i < polls; ++i) {
        if (mbar_try_wait(bar, parity)) { ok = true; break; }
        if ((i & 255u) == 255u && sh->abort) break;
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) sh->abort = 1;
    return ok;
}

// At most 88 registers: next to the streaming kernel's CTA (8 warps of 168 registers, two per scheduler) a
// scheduler's 16,384 registers leave room for two of this kernel's warps only up to that size.
template <int D>
__global__ void __maxnreg__(88) attn_partial_wide_kernel(DecodeArgs a, int first_item) {
    constexpr uint32_t TB = 16 * D * 2;                  // one tile
    constexpr uint32_t STAGE_HALF = kStageUnits * TB;    // K (or V) part of a stage
    constexpr int KS = D / 16;                           // k-steps of the QK product
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    uint8_t* base_ptr = smem_raw;
    const uint32_t q_smem = base;                                     // 128 rows x D bf16
    const uint32_t ring = base + 128u * D * 2u;                       // kStages x (K half, V half)
    Shared* sh = reinterpret_cast<Shared*>(base_ptr + 128u * D * 2u + kStages * 2u * STAGE_HALF);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Launch order (see pdl_wait in ets_device.cuh).  The merge kernel behind this one may become resident
    // at once; it waits for this kernel to complete before it reads a partial result.  Launched on its own,
    // this kernel waits here for the kernel ahead of it (an append, or the previous call's merge) before it
    // reads lengths, K/V or queries.  Launched behind the narrow kernel of the same call it must not: that
    // wait would last until the narrow kernel has finished, and the two are meant to share the SMs.  It
    // needs none then: the narrow kernel lets it start only after its own wait, i.e. when everything
    // earlier in the stream has completed.  Completion stays transitive because the CTA that finishes
    // last waits for the narrow kernel before it leaves (at the end of this function).
    unsigned int stamp = 0;
    if (a.stamps && threadIdx.x == 0) stamp = stamp_start(a.stamps, 2);
    pdl_launch_dependents();
    if (!a.wide_behind_narrow) pdl_wait();
    if (base & 1023u) {   // the swizzled operand layout needs 1024-byte aligned tiles
        if (threadIdx.x == 0) atomicExch(a.status, -1);
        pdl_wait();
        return;
    }
    const DevItem it = a.items[first_item + blockIdx.x];
    const int G = a.G, h = it.kv_head;
    const int rows = it.n_leaves_tile * G;

    // Producer step, K part: take the next page slots of the item that hold tokens (up to kStageUnits),
    // describe stage st in info[st % kInfoRing], start the copies of their K tiles into stage st % kStages and
    // publish.  Returns the number of slots (0 = end marker).  Called by all lanes of warp 0.  The descriptors
    // of 32 consecutive page slots, one per lane, are kept in registers between calls: the two dependent table
    // loads behind them are paid once per 32 slots, not once per stage.
    int u = 0, win_base = -32;
    int w_page = 0, w_valid = 0, w_node = -1, w_tok0 = 0;
    uint32_t w_live = 0;
    uint32_t prod_k = 0, prod_v = 0;   // stages whose K / V copies were started
    auto produce_k = [&](uint32_t st) -> int {
        const uint32_t s = st % kStages;
        StageInfo* inf = &sh->info[st % kInfoRing];
        int n = 0;
        int my_pg = 0, my_vl = 0, my_nd = -1, my_t0 = 0;
        const uint32_t kdst = ring + s * 2 * STAGE_HALF;
        while (n < kStageUnits && u < it.unit_count) {
            if (u >= win_base + 32) {
                win_base = u;
                const int idx = u + lane;
                w_page = 0; w_valid = 0; w_node = -1; w_tok0 = 0;
                if (idx < it.unit_count) {
                    const int4 un = a.units[it.unit_begin + idx];
                    w_node = un.y;
                    w_tok0 = un.z;
                    w_valid = a.node_len[un.y] - un.z;
                    w_valid = w_valid < 0 ? 0 : (w_valid > 16 ? 16 : w_valid);
                    if (w_valid > 0 && (un.x < 0 || (int64_t)un.x >= a.pages_per_layer)) { atomicExch(a.status, -1); w_valid = 0; }
                    w_page = un.x;
                }
                w_live = __ballot_sync(0xffffffffu, w_valid > 0);
            }
            const uint32_t rest = w_live >> (u - win_base);      // live slots of the window from u on
            if (rest == 0) { u = win_base + 32; continue; }
            const int src = (u - win_base) + __ffs(rest) - 1;
            u = win_base + src + 1;
            const int pg = __shfl_sync(0xffffffffu, w_page, src);
            const int vl = __shfl_sync(0xffffffffu, w_valid, src);
            const int nd = __shfl_sync(0xffffffffu, w_node, src);
            const int t0 = __shfl_sync(0xffffffffu, w_tok0, src);
            if (lane == n) { my_pg = pg; my_vl = vl; my_nd = nd; my_t0 = t0; }   // lane n: the slot's copies
            ++n;
        }
        // All copies of the half stage are started by one instruction, one lane per tile (a bulk copy occupies
        // the lane that starts it for some hundred cycles).  The byte count is raised first; the producer's
        // single arrival comes after the copies have been started, so the phase cannot end early.
        if (lane == 0 && n > 0)
            asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&sh->full_k[s])), "r"((uint32_t)n * TB) : "memory");
        __syncwarp();
        if (lane < n) {
            inf->page[lane] = my_pg;
            inf->valid[lane] = my_vl;
            inf->node[lane] = my_nd;
            inf->tok0[lane] = my_t0;
            bulk_g2s(kdst + lane * TB, kv_tile(a.k_pool, a.v_pool, a.pages_per_layer, my_pg, h, TB), TB, smem_u32(&sh->full_k[s]));
        }
        __syncwarp();
        if (u > it.unit_count) u = it.unit_count;
        if (lane == 0) {
            inf->n_units = n;                         // n == 0: end marker
            mbar_arrive(smem_u32(&sh->full_k[s]));    // publishes the stage info with release semantics
        }
        __syncwarp();
        if (n > 0) ++prod_k;
        return n;
    };
    // V part of a stage that produce_k described: its V tiles follow the K tiles in the page image.
    auto produce_v = [&](uint32_t st) {
        const uint32_t s = st % kStages;
        const StageInfo* inf = &sh->info[st % kInfoRing];
        const int n = inf->n_units;
        const uint32_t vdst = ring + s * 2 * STAGE_HALF + STAGE_HALF;
        if (lane == 0)
            asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&sh->full_v[s])), "r"((uint32_t)n * TB) : "memory");
        __syncwarp();
        if (lane < n)
            bulk_g2s(vdst + lane * TB, kv_tile(a.k_pool, a.v_pool, a.pages_per_layer, inf->page[lane], h, TB) + TB, TB, smem_u32(&sh->full_v[s]));
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh->full_v[s]));
        __syncwarp();
        ++prod_v;
    };

    int n_first = 0;
    if (warp == 0) {
        if (lane == 0) {
            for (int s = 0; s < kStages; ++s) {
                mbar_init(smem_u32(&sh->full_k[s]), 1);
                mbar_init(smem_u32(&sh->full_v[s]), 1);
                mbar_init(smem_u32(&sh->empty_k[s]), 1);
                mbar_init(smem_u32(&sh->empty_v[s]), 1);
            }
            mbar_init(smem_u32(&sh->s_ready[0]), 1);
            mbar_init(smem_u32(&sh->s_ready[1]), 1);
            mbar_init(smem_u32(&sh->p_ready), 4);
            mbar_init(smem_u32(&sh->o_ready), 1);
            sh->abort = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        // the first stage's copies start before anybody else is ready for them
        n_first = produce_k(0);
        if (n_first > 0) produce_v(0);
    } else {
        // Q tile: query row r = (leaf r / G of the tile, head h*G + r % G), K-major with the 128-byte
        // swizzle.  The producer warp is already fetching K/V meanwhile.  Leaf ids are fetched once
        // per warp and all of a thread's 16-byte loads are issued before the first store, so the
        // gather costs two memory round trips instead of two per chunk.
        constexpr int kGatherThreads = kWideThreads - 32;
        constexpr int kPer = (128 * (D / 8) + kGatherThreads - 1) / kGatherThreads;
        const int my_leaf = lane < it.n_leaves_tile ? a.node_leaves[it.leaf_list_begin + lane] : 0;
        const int leaf_hi = (lane + 32 < it.n_leaves_tile) ? a.node_leaves[it.leaf_list_begin + lane + 32] : 0;
        const int leaf_h2 = (lane + 64 < it.n_leaves_tile) ? a.node_leaves[it.leaf_list_begin + lane + 64] : 0;
        const int leaf_h3 = (lane + 96 < it.n_leaves_tile) ? a.node_leaves[it.leaf_list_begin + lane + 96] : 0;
        constexpr int kBatch = kPer;   // all of a thread's loads in flight at once: the roles' registers are not live yet
#pragma unroll 1
        for (int k0 = 0; k0 < kPer; k0 += kBatch) {
            uint4 v[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int i = (int)threadIdx.x - 32 + (k0 + k) * kGatherThreads;
                const int r = i / (D / 8), c = i % (D / 8);
                const int lr = r / G;                       // leaf of the tile (up to 128 when G = 1)
                const int l0 = __shfl_sync(0xffffffffu, my_leaf, lr & 31);
                const int l1 = __shfl_sync(0xffffffffu, leaf_hi, lr & 31);
                const int l2 = __shfl_sync(0xffffffffu, leaf_h2, lr & 31);
                const int l3 = __shfl_sync(0xffffffffu, leaf_h3, lr & 31);
                const int leaf = lr < 32 ? l0 : (lr < 64 ? l1 : (lr < 96 ? l2 : l3));
                v[k] = make_uint4(0u, 0u, 0u, 0u);
                if (i < 128 * (D / 8) && r < rows)
                    v[k] = __ldg(reinterpret_cast<const uint4*>(a.q + ((size_t)leaf * a.Hq + h * G + r % G) * D + c * 8));
            }
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int i = (int)threadIdx.x - 32 + (k0 + k) * kGatherThreads;
                if (i < 128 * (D / 8)) *reinterpret_cast<uint4*>(base_ptr + tile_offset(D, i / (D / 8), (i % (D / 8)) * 8)) = v[k];
            }
        }
        fence_proxy_async();      // the Q tile was written by ordinary stores and is read by the MMA unit
    }
    tc_fence_before();
    asm volatile("bar.sync 1, %0;" ::"r"(kWideThreads) : "memory");   // barriers, TMEM address, Q tile: visible to all
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        // Order of the copies: K0 V0 K1 V1 K2, then K(j+1), V(j) for j = 2, 3, ...: a K half is refilled when
        // the product that read it has run, which is a whole stage before the V half of the same stage is free.
        if (n_first > 0 && produce_k(1) > 0) {
            produce_v(1);
            int n_next = 0;
            if (wait_or_abort(smem_u32(&sh->empty_k[0]), 0u, sh)) n_next = produce_k(2);            // QK(0) has run
            for (uint32_t j = 2; n_next > 0; ++j) {    // stage j: K on its way, V not yet
                if (!wait_or_abort(smem_u32(&sh->empty_k[(j + 1) % kStages]), (((j + 1) / kStages) - 1) & 1u, sh)) break;   // QK(j - 1)
                n_next = produce_k(j + 1);
                if (!wait_or_abort(smem_u32(&sh->empty_v[j % kStages]), ((j / kStages) - 1) & 1u, sh)) break;               // PV(j - 2)
                produce_v(j);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc_pv = instr_desc(D, true);
        // S = Q K^T of stage st into S buffer st % 2 (or the end marker); returns the stage's page slots, -1 on abort
        auto issue_qk = [&](uint32_t st) -> int {
            const uint32_t s = st % kStages;
            if (!wait_or_abort(smem_u32(&sh->full_k[s]), (st / kStages) & 1u, sh, st == 0 ? a.first_wait_polls : kSpin)) return -1;
            const int n = sh->info[st % kInfoRing].n_units;
            if (n == 0) {   // end of item: wake the softmax warps, which then see the same marker
                if (lane == 0) mbar_arrive(smem_u32(&sh->s_ready[st & 1u]));
                return 0;
            }
            const uint32_t kst = ring + s * 2 * STAGE_HALF;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t idesc_qk = instr_desc(16u * n, false);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const uint32_t koff = (uint32_t)(ks >> 2) * 1024u + (uint32_t)(ks & 3) * 32u;
                    umma_ss(tmem + kColS + kColSBuf * (st & 1u), smem_desc(q_smem + koff, 16, 1024u * (D / 64)),
                            smem_desc(kst + koff, 16, 1024u * (D / 64)), idesc_qk, ks > 0);
                }
                umma_commit(smem_u32(&sh->s_ready[st & 1u]));
                umma_commit(smem_u32(&sh->empty_k[s]));
            }
            __syncwarp();
            return n;
        };
        // The S buffer of stage st + 2 held S and P of stage st, whose second product was issued by this
        // thread just before: the tensor pipe runs a thread's products in order, so the buffer is free by then.
        int n = issue_qk(0);
        int n_next = n > 0 ? issue_qk(1) : 0;
        for (uint32_t st = 0; n > 0 && n_next >= 0; ++st) {
            const uint32_t s = st % kStages;
            const StageInfo* inf = &sh->info[st % kInfoRing];
            const uint32_t vst = ring + s * 2 * STAGE_HALF + STAGE_HALF;
            if (!wait_or_abort(smem_u32(&sh->full_v[s]), (st / kStages) & 1u, sh)) break;
            // rows past a page's length hold stale bytes; zero them in V (0 * garbage could be NaN)
            bool wrote = false;
            for (int k = 0; k < n; ++k) {
                const int valid = inf->valid[k];
                if (valid < 16) {
                    for (int i = lane; i < (16 - valid) * (D / 8); i += 32) {
                        const int t = valid + i / (D / 8), c = i % (D / 8);
                        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vst + k * TB + tile_offset(D, t, c * 8)), "r"(0u) : "memory");
                    }
                    wrote = true;
                }
            }
            if (wrote) fence_proxy_async();
            __syncwarp();
            if (!wait_or_abort(smem_u32(&sh->p_ready), st & 1u, sh)) break;
            tc_fence_after();
            if (lane == 0) {
                for (int k = 0; k < n; ++k)
                    umma_ts(tmem + kColO, tmem + kColP + kColSBuf * (st & 1u) + p_col(k), smem_desc(vst + k * TB, 1024, 1024u * (D / 64)),
                            idesc_pv, !(st == 0 && k == 0));
                // the weights' second term
                for (int k = 0; k < n; ++k)
                    umma_ts(tmem + kColO, tmem + kColP + kColPLo + kColSBuf * (st & 1u) + p_col(k), smem_desc(vst + k * TB, 1024, 1024u * (D / 64)),
                            idesc_pv, true);
                umma_commit(smem_u32(&sh->empty_v[s]));
                umma_commit(smem_u32(&sh->o_ready));
            }
            __syncwarp();
            int n_after = 0;
            if (n_next > 0) n_after = issue_qk(st + 2);
            n = n_next;
            n_next = n_after;
        }
    } else {
        // ------------------------------------------------------------------ softmax, one row per thread
        const int row = 32 * (warp & 3) + lane;
        const uint32_t tlane = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
        float m_ref = -INFINITY, l = 0.f;
        uint32_t n_stages = 0;
        bool ok = true;
        // step prefill: this row's query sees only the first `lim` tokens of the node it sits at
        int own_node = -1, lim = 0;
        if (a.leaf_limit != nullptr && row < rows) {
            const int leaf = a.node_leaves[it.leaf_list_begin + row / G];
            own_node = a.leaf_node[leaf];
            lim = a.leaf_limit[leaf];
        }
        auto row_valid = [&](uint32_t s, int c) {
            int v = sh->info[s].valid[c];
            if (sh->info[s].node[c] == own_node) {
                const int x = lim - sh->info[s].tok0[c];
                v = x < v ? (x < 0 ? 0 : x) : v;
            }
            return v;
        };
        for (uint32_t st = 0;; ++st) {
            const uint32_t s = st % kInfoRing;
            if (!wait_or_abort(smem_u32(&sh->s_ready[st & 1u]), (st >> 1) & 1u, sh)) { ok = false; break; }
            // s_ready can only complete after the MMA warp saw full_k of the stage: the stage info is visible
            const int n = sh->info[s].n_units;
            if (n == 0) break;   // end marker passed on by the MMA warp
            tc_fence_after();
            // pass 1: row maximum over the stage's tokens, two page slots (32 columns) per load; for
            // an odd count the last load also reads 16 stale S columns, which are masked
            float mx = -INFINITY;
            for (int c = 0; c < n; c += 2) {
                float v[32];
                tmem_ld32(tlane + kColS + kColSBuf * (st & 1u) + 16u * c, v);
                const int v0 = row_valid(s, c);
                const int v1 = c + 1 < n ? row_valid(s, c + 1) : 0;
                float m0 = -INFINITY, m1 = -INFINITY;
                if (v0 == 16 && v1 == 16) {   // two full pages, the usual case: no per-token test
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        m0 = max3(m0, v[i], v[i + 1]);
                        m1 = max3(m1, v[16 + i], v[16 + i + 1]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        if (i < v0) m0 = fmaxf(m0, v[i]);
                        if (i < v1) m1 = fmaxf(m1, v[16 + i]);
                    }
                }
                mx = fmaxf(mx, fmaxf(m0, m1));
            }
            mx *= a.scale_log2;
            // O must hold the previous stage's product before it is rescaled, and that product must have read
            // its P before this stage's P is handed over: wait for it here, after the maximum pass, which
            // thereby overlaps the product
            if (st > 0) {
                if (!wait_or_abort(smem_u32(&sh->o_ready), (st - 1) & 1u, sh)) { ok = false; break; }
                tc_fence_after();
            }
            // raise the reference (and rescale O, l) when the maximum outgrew it by the threshold
            const bool need = mx > m_ref + kRescaleThreshold;
            const bool any_need = __any_sync(0xffffffffu, need);
            if (any_need) {
                const float m_new = need ? mx : m_ref;
                const float f = (m_ref == -INFINITY) ? 0.f : exp2f(m_ref - m_new);
                if (st > 0) {
                    // O of the previous stages is final in tensor memory (o_ready was waited for below)
#pragma unroll 1
                    for (int c = 0; c < D; c += 32) {
                        float v[32];
                        tmem_ld32(tlane + kColO + c, v);
                        const float2 f2 = make_float2(f, f);
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {   // packed fp32 multiplies: half the instructions
                            const float2 r = __fmul2_rn(make_float2(v[i], v[i + 1]), f2);
                            v[i] = r.x;
                            v[i + 1] = r.y;
                        }
                        tmem_st32(tlane + kColO + c, v);
                    }
                    tmem_wait_st();
                }
                l *= f;
                m_ref = m_new;
            }
            // pass 2: P = 2^(s - m_ref), packed bf16 into the A operand of the second product, two page
            // slots per step with independent sums.  A weight goes in as two bf16 terms, its rounded
            // value and the rounded rest: with one term the weights would be off by up to 2^-8 each,
            // which on a path of a few tokens with values of opposite sign exceeds the output's
            // tolerance.  Both terms of a pair go where the pair's S was.
            // The scaling, the rests and the row sums use the packed fp32 instructions (two lanes per
            // instruction): the softmax warps are bound by the number of instructions they issue.
            float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
            const float2 sc2 = make_float2(a.scale_log2, a.scale_log2), nr2 = make_float2(-m_ref, -m_ref);
            const float2 minus1 = make_float2(-1.f, -1.f);
            for (int c = 0; c < n; c += 2) {
                float v[32];
                tmem_ld32(tlane + kColS + kColSBuf * (st & 1u) + 16u * c, v);
                const int v0 = row_valid(s, c);
                const int v1 = c + 1 < n ? row_valid(s, c + 1) : 0;
                uint32_t pk[16], plo[16];
                const bool full = v0 == 16 && v1 == 16;
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    // weights are at most 1 and are rounded to bf16 next: the approximate exponential
                    // (2 ulp, tiny results flushed to zero) loses nothing
                    const float2 xa = __ffma2_rn(make_float2(v[i], v[i + 1]), sc2, nr2);
                    const float2 xb = __ffma2_rn(make_float2(v[16 + i], v[16 + i + 1]), sc2, nr2);
                    float2 wa, wb;
                    wa.x = (full || i < v0) ? ex2_approx(xa.x) : 0.f;
                    wa.y = (full || i + 1 < v0) ? ex2_approx(xa.y) : 0.f;
                    wb.x = (full || i < v1) ? ex2_approx(xb.x) : 0.f;
                    wb.y = (full || i + 1 < v1) ? ex2_approx(xb.y) : 0.f;
                    const __nv_bfloat162 pa = __floats2bfloat162_rn(wa.x, wa.y);
                    const __nv_bfloat162 pb = __floats2bfloat162_rn(wb.x, wb.y);
                    // rest = weight - rounded weight (exact in fp32)
                    const float2 ra = __ffma2_rn(make_float2(__low2float(pa), __high2float(pa)), minus1, wa);
                    const float2 rb = __ffma2_rn(make_float2(__low2float(pb), __high2float(pb)), minus1, wb);
                    const __nv_bfloat162 qa = __floats2bfloat162_rn(ra.x, ra.y);
                    const __nv_bfloat162 qb = __floats2bfloat162_rn(rb.x, rb.y);
                    la = __fadd2_rn(la, wa);
                    lb = __fadd2_rn(lb, wb);
                    pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&pa);
                    pk[8 + (i >> 1)] = *reinterpret_cast<const uint32_t*>(&pb);
                    plo[i >> 1] = *reinterpret_cast<const uint32_t*>(&qa);
                    plo[8 + (i >> 1)] = *reinterpret_cast<const uint32_t*>(&qb);
                }
                tmem_st16(tlane + kColP + kColSBuf * (st & 1u) + p_col(c), pk);
                tmem_st16(tlane + kColP + kColPLo + kColSBuf * (st & 1u) + p_col(c), plo);
            }
            const float l0 = la.x + la.y, l1 = lb.x + lb.y;
            l += l0 + l1;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->p_ready));
            ++n_stages;
        }
        // the last stage's product must be in O before the epilogue reads it
        if (ok && n_stages > 0) {
            if (!wait_or_abort(smem_u32(&sh->o_ready), (n_stages - 1) & 1u, sh)) ok = false;
            tc_fence_after();
        }
        // epilogue: partial (m_ref, l, O) of this row
        if (ok && row < rows) {
            const size_t prow = (size_t)(it.slot_first + row / G) * G + row % G;
            a.part_ml[prow] = make_float2(m_ref, l);
        }
        if (ok) {
            // O goes out through shared memory: a thread owns a row, so stores straight from its registers would
            // touch 32 different 512-byte rows per instruction.  Each thread lays its row down in the (now idle)
            // Q tile and K/V ring, rows 16 bytes apart from a multiple of 512 so that the 16-byte stores of a
            // warp spread over all banks, and sends it with one bulk copy.  Nothing else uses that memory any
            // more: the wait for the last product above covers every product of this CTA, and every copy that
            // was started has been consumed by one of them.
            constexpr uint32_t kRowBytes = D * 4 + 16;
            static_assert(128u * kRowBytes <= 128u * D * 2u + kStages * 2u * STAGE_HALF, "O staging fits in the Q tile and the ring");
            const uint32_t row_smem = base + (uint32_t)row * kRowBytes;
            float* po = a.part_o + ((size_t)(it.slot_first + row / G) * G + row % G) * D;
#pragma unroll 1
            for (int c = 0; c < D; c += 32) {
                float v[32];
                if (n_stages > 0) tmem_ld32(tlane + kColO + c, v);
                else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(row_smem + (uint32_t)(c + i) * 4u), "f"(v[i]), "f"(v[i + 1]),
                                 "f"(v[i + 2]), "f"(v[i + 3])
                                 : "memory");
            }
            if (row < rows) {
                fence_proxy_async();   // the row was written by ordinary stores and is read by the copy engine
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(po), "r"(row_smem), "r"((uint32_t)(D * 4)) : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // own copy only; it reads this CTA's shared memory
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (sh->abort) {
        if (threadIdx.x == 0) atomicExch(a.status, -7);
        // copies that were started still target this CTA's shared memory: give them time to land
        if (warp == 0) {
            for (uint32_t st = prod_k > (uint32_t)kStages ? prod_k - kStages : 0u; st < prod_k; ++st) {
                const uint32_t bar = smem_u32(&sh->full_k[st % kStages]), par = (st / kStages) & 1u;
                for (uint32_t i = 0; i < kSpin && !mbar_try_wait(bar, par); ++i) {}
            }
            for (uint32_t st = prod_v > (uint32_t)kStages ? prod_v - kStages : 0u; st < prod_v; ++st) {
                const uint32_t bar = smem_u32(&sh->full_v[st % kStages]), par = (st / kStages) & 1u;
                for (uint32_t i = 0; i < kSpin && !mbar_try_wait(bar, par); ++i) {}
            }
        }
        __syncthreads();
    }
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    // behind the narrow kernel: the CTA that finishes last waits for that kernel, so that this grid
    // completes after it (the others leave at once and free their SM for the CTAs still queued)
    if (a.stamps && threadIdx.x == 0) stamp_end(a.stamps, 2, stamp, gridDim.x);
    if (a.wide_behind_narrow && threadIdx.x == 0) {
        if (atomicAdd(a.queue + 2, 1) == (int)gridDim.x - 1) {
            a.queue[2] = 0;
            pdl_wait();
        }
    }
}

size_t wide_smem_bytes_impl(int D) {
    return 128u * D * 2u + kStages * 2u * kStageUnits * 16u * D * 2u + sizeof(Shared) + 64;
}

}  // namespace

size_t wide_smem_bytes(int D) { return wide_smem_bytes_impl(D); }

cudaError_t wide_prepare(int D) {
    // the largest shared-memory carve-out, so that a CTA of the other attention kernel can be
    // resident on the same SM
    cudaError_t e;
    if (D == 128) {
        e = cudaFuncSetAttribute(attn_partial_wide_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)wide_smem_bytes_impl(128));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_partial_wide_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    } else {
        e = cudaFuncSetAttribute(attn_partial_wide_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)wide_smem_bytes_impl(64));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_partial_wide_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    }
    return e;
}

void launch_partial_wide(const DecodeArgs& a, int D, int first_item, int n_wide, bool chained, cudaStream_t s) {
    if (n_wide <= 0) return;
    ChainLaunch l(dim3(n_wide), dim3(kWideThreads), wide_smem_bytes_impl(D), s, chained);
    if (D == 128) cudaLaunchKernelEx(&l.cfg, attn_partial_wide_kernel<128>, a, first_item);
    else cudaLaunchKernelEx(&l.cfg, attn_partial_wide_kernel<64>, a, first_item);
}

}  // namespace ets
