// Log-sum-exp merge of the partials of one (leaf, query head), by one warp.
//
// With partials (m_j, l_j, o_j) in log2 units over disjoint token blocks:
//   m* = max_j m_j, l* = sum_j l_j 2^(m_j-m*), out = sum_j o_j 2^(m_j-m*) / l*,
//   lse = (m* + log2 l*) ln 2.
// Empty partials (l_j = 0) are skipped; a row without any token gives zeros and lse = -inf.
// This is the exact softmax of the union of the blocks.
#pragma once
#include "ets_device.cuh"

namespace ets {

// One (leaf, query head) per warp.  Lanes fetch the slot ids and then the (m, l) pairs in parallel;
// after that the addresses of all o rows are known and their loads do not depend on each other.
// The partial slots of one (leaf, query head): bounds of its list and this lane's entry of the first 32.
// Read from the tables only, so a caller may fetch it before the partial results exist.
struct MergeList {
    int s0, s1, first_slot;
};
__device__ __forceinline__ MergeList merge_list(const DecodeArgs& a, int leaf, int head, int lane) {
    MergeList m;
    const int list = leaf * a.Hkv + head / a.G;
    m.s0 = a.leaf_slot_off[list];
    m.s1 = a.leaf_slot_off[list + 1];
    m.first_slot = m.s0 + lane < m.s1 ? a.leaf_slots[m.s0 + lane] : -1;
    return m;
}

// kEarly: o rows whose loads are started together with the (m, l) loads (registers: kEarly * D / 32)
template <int D, int kEarly = 8>
__device__ __forceinline__ void merge_row(const DecodeArgs& a, int leaf, int head, int lane, const MergeList& list) {
    constexpr int EPL = D / 32;  // features per lane
    const int G = a.G, sub = head % G;
    const int s0 = list.s0, s1 = list.s1;
    float ms = -INFINITY, ls = 0.f;
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int base = s0; base < s1; base += 32) {
        const int cnt = min(32, s1 - base);
        const int my_slot = base == s0 ? list.first_slot : (lane < cnt ? a.leaf_slots[base + lane] : -1);
        float2 ml = make_float2(-INFINITY, 0.f);
        if (my_slot >= 0) ml = a.part_ml[(size_t)my_slot * G + sub];
        // the addresses of the o rows depend on the slot ids only: start the first loads now, so that
        // they travel together with the (m, l) pairs instead of after the reduction over them
        float early[kEarly][EPL];
#pragma unroll
        for (int j = 0; j < kEarly; ++j) {
            const int slot = __shfl_sync(0xffffffffu, my_slot, j);
#pragma unroll
            for (int e = 0; e < EPL; ++e) early[j][e] = 0.f;
            if (j < cnt) {
                const float* po = a.part_o + ((size_t)slot * G + sub) * D + lane * EPL;
                if constexpr (EPL == 4) {
                    const float4 v = *reinterpret_cast<const float4*>(po);
                    early[j][0] = v.x; early[j][1] = v.y; early[j][2] = v.z; early[j][3] = v.w;
                } else {
                    const float2 v = *reinterpret_cast<const float2*>(po);
                    early[j][0] = v.x; early[j][1] = v.y;
                }
            }
        }
        float bm = ml.y > 0.f ? ml.x : -INFINITY;
#pragma unroll
        for (int x = 16; x > 0; x >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, x));
        const float mn = fmaxf(ms, bm);
        const float corr = mn > -INFINITY ? exp2f(ms - mn) : 0.f;
        const float wgt = ml.y > 0.f ? exp2f(ml.x - mn) : 0.f;
        float wl = wgt * ml.y;
#pragma unroll
        for (int x = 16; x > 0; x >>= 1) wl += __shfl_xor_sync(0xffffffffu, wl, x);
        ls = ls * corr + wl;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] *= corr;
        ms = mn;
#pragma unroll
        for (int j = 0; j < kEarly; ++j) {
            const float w = __shfl_sync(0xffffffffu, wgt, j);
            if (j < cnt && w > 0.f) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[e] += w * early[j][e];
            }
        }
#pragma unroll 8
        for (int j = kEarly; j < cnt; ++j) {
            const int slot = __shfl_sync(0xffffffffu, my_slot, j);
            const float w = __shfl_sync(0xffffffffu, wgt, j);
            const float* po = a.part_o + ((size_t)slot * G + sub) * D + lane * EPL;
            if constexpr (EPL == 4) {
                const float4 v = *reinterpret_cast<const float4*>(po);
                if (w > 0.f) { acc[0] += w * v.x; acc[1] += w * v.y; acc[2] += w * v.z; acc[3] += w * v.w; }
            } else {
                const float2 v = *reinterpret_cast<const float2*>(po);
                if (w > 0.f) { acc[0] += w * v.x; acc[1] += w * v.y; }
            }
        }
    }
    const float inv = ls > 0.f ? 1.f / ls : 0.f;
    const size_t row = (size_t)leaf * a.Hq + head;
    __nv_bfloat16* op = a.out + row * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; e += 2)
        *reinterpret_cast<__nv_bfloat162*>(op + e) = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
    if (a.lse && lane == 0) a.lse[row] = ls > 0.f ? (ms + log2f(ls)) * 0.6931471805599453f : -INFINITY;
}

}  // namespace ets
