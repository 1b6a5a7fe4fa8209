// Measurement probes (no step of the method): what this GPU gives a kernel shaped like the streaming
// attention kernel when all arithmetic is taken away, and what a launch costs.  bench.py reports them next
// to the attention kernels' numbers; nothing else uses them.
#include "../../include/ets.h"

#include <cuda_runtime.h>
#include <cstdint>

namespace {

constexpr int kProbeWarps = 8;
constexpr uint32_t kProbePolls = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Persistent grid, kProbeWarps independent warps per CTA, each with a ring of `depth` shared-memory slots
// of `chunk` bytes filled by linear bulk copies that complete on the slot's mbarrier: the narrow attention
// kernel's data path and nothing else.  Chunk i of the buffer goes to warp i % n_warps.  Every lane reads one
// word of each chunk that lands (so the data is really consumed) and the xor of all of them is stored once.
__global__ void __launch_bounds__(kProbeWarps * 32) stream_read_kernel(const char* buf, int64_t n_chunks, uint32_t chunk,
                                                                     int depth, uint32_t* sink, int32_t* status) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * kProbeWarps;
    const int64_t me = (int64_t)blockIdx.x * kProbeWarps + warp;
    const uint32_t ring = base + (uint32_t)warp * depth * chunk;
    const uint32_t bars = base + (uint32_t)kProbeWarps * depth * chunk + (uint32_t)warp * depth * 8;
    if (lane == 0) {
        for (int s = 0; s < depth; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bars + s * 8), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const int64_t mine = me < n_chunks ? (n_chunks - me + n_warps - 1) / n_warps : 0;
    int64_t issued = 0, consumed = 0;
    uint32_t acc = 0;
    bool dead = false;
    auto issue = [&]() {
        if (lane == 0) {
            const uint32_t slot = (uint32_t)(issued % depth);
            const char* src = buf + (size_t)(me + issued * n_warps) * chunk;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bars + slot * 8), "r"(chunk) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(ring + slot * chunk),
                         "l"(src), "r"(chunk), "r"(bars + slot * 8)
                         : "memory");
        }
        ++issued;
    };
    auto wait = [&](int64_t k) {
        const uint32_t bar = bars + (uint32_t)(k % depth) * 8, parity = (uint32_t)((k / depth) & 1);
        bool ok = false;
        for (uint32_t i = 0; i < kProbePolls && !ok; ++i) {
            uint32_t r;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(r) : "r"(bar), "r"(parity) : "memory");
            ok = r != 0;
        }
        return __all_sync(0xffffffffu, ok);
    };
    while (issued < mine && issued < depth) issue();
    while (consumed < mine && !dead) {
        if (!wait(consumed)) { dead = true; break; }
        uint32_t w;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(ring + (uint32_t)(consumed % depth) * chunk + (uint32_t)lane * 4u) : "memory");
        acc ^= w;
        ++consumed;
        __syncwarp();
        if (issued < mine) issue();
    }
    if (dead) {   // a wait ran out: flag it, let the copies in flight land, leave
        if (lane == 0) atomicExch(status, -7);
        ++consumed;
        while (consumed < issued) { wait(consumed); ++consumed; }
    }
    if (acc == 0x9e3779b9u) sink[me & 1023] = acc;   // keeps the loads alive; practically never taken
}

__global__ void __launch_bounds__(kProbeWarps * 32) empty_kernel(int32_t*) {}

}  // namespace

extern "C" {

int32_t ets_probe_stream_read(const void* buf, size_t bytes, int32_t chunk_bytes, int32_t depth, int32_t n_ctas,
                              void* scratch, void* cuda_stream) {
    if (!buf || !scratch || chunk_bytes < 1024 || chunk_bytes % 1024 || depth < 1 || depth > 8 || n_ctas < 1)
        return ETS_ERR_INVALID_ARG;
    if (((uintptr_t)buf & 1023) || ((uintptr_t)scratch & 15)) return ETS_ERR_INVALID_ARG;
    const size_t smem = (size_t)kProbeWarps * depth * chunk_bytes + kProbeWarps * depth * 8;
    if (smem > 227 * 1024) return ETS_ERR_INVALID_ARG;
    if (cudaFuncSetAttribute(stream_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return ETS_ERR_CUDA;
    const int64_t n_chunks = (int64_t)(bytes / (size_t)chunk_bytes);
    uint32_t* sink = reinterpret_cast<uint32_t*>(scratch);
    int32_t* status = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(scratch) + 4096);
    stream_read_kernel<<<n_ctas, kProbeWarps * 32, smem, (cudaStream_t)cuda_stream>>>((const char*)buf, n_chunks, (uint32_t)chunk_bytes,
                                                                                   depth, sink, status);
    return cudaGetLastError() == cudaSuccess ? ETS_OK : ETS_ERR_CUDA;
}

int32_t ets_probe_empty_launch(int32_t n_ctas, size_t smem_bytes, void* scratch, void* cuda_stream) {
    if (n_ctas < 1 || smem_bytes > 227 * 1024 || !scratch) return ETS_ERR_INVALID_ARG;
    static size_t allowed = 0;   // raise the kernel's shared-memory limit only when a call needs more than before
    if (smem_bytes > allowed) {
        if (cudaFuncSetAttribute(empty_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
            return ETS_ERR_CUDA;
        allowed = smem_bytes;
    }
    empty_kernel<<<n_ctas, kProbeWarps * 32, smem_bytes, (cudaStream_t)cuda_stream>>>(reinterpret_cast<int32_t*>(scratch));
    return cudaGetLastError() == cudaSuccess ? ETS_OK : ETS_ERR_CUDA;
}

}  // extern "C"
