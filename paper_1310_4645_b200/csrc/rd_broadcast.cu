// sm_100a kernels of the broadcast that turns a reduce into an all-reduce (Section III: an all-reduce is a
// reduce followed by a broadcast of the root's result).
//
// The broadcast moves m bytes in and n_dst * m bytes out, so it is bound by HBM writes and has no arithmetic at
// all.  Two kernels, chosen by the number of destinations (measured on 64 MiB messages, both on one B200, time of the
// broadcast alone in microseconds, bulk copies / registers: 1 destination 17 / 19, 7: 102 / 105, 15: 199 / 204,
// 31: 383 / 377, 63: 769 / 727, 255: 2898 / 2753):
//   rd_broadcast_bulk_kernel   up to kBulkMostDst destinations, every buffer 16-byte aligned.  No data in registers:
//                              one thread per thread block brings a tile of the source into shared memory with one
//                              bulk asynchronous copy and sends it to every destination with one bulk asynchronous
//                              copy each (cp.async.bulk, shared -> global); tiles go round robin over the thread
//                              blocks, several small thread blocks per SM keep enough bytes in flight.
//   rd_broadcast_kernel<V>     every thread carries kU vectors of V words from the source to each destination:
//                              V = 4 for aligned buffers and many destinations, V = 1 for buffers that are not
//                              16-byte aligned and for the last n mod 4 words.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "rd_kernels.h"

namespace rd {

namespace {

constexpr int kThreads = 256;
constexpr int kU = 4;                                   // vectors in flight per thread
constexpr long long kWaitCycles = 4000000000ll;         // a wait gives up after about two seconds of SM clock
// Ring of the bulk-copy kernel: 4 KB stages, eight per thread block, so seven thread blocks per SM.  Measured on
// 64 MiB messages: 2 KB ... 16 KB stages with 32 KB per thread block are within 3 % of each other, which is what two
// runs of one shape differ by; 512-byte stages and rings of 8 KB are 3-8 % behind.
constexpr int kBulkTile = 4096;
constexpr int kBulkStages = 8;
constexpr int kBulkMostDst = 16;
constexpr int kDevices = 64;

struct BcastParams {
    uint32_t *dst[kBcastPackPtrs];
    const uint32_t *src;
    uint64_t n;                          // bytes (bulk kernel) or vectors of V words (register kernel) to copy
    int n_dst;
    int *status;                         // device word: 0, or the first error code
};

template <int V>
__global__ void __launch_bounds__(kThreads, 4)
rd_broadcast_kernel(const __grid_constant__ BcastParams a)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");           // the reduction that produced src has finished
    const uint64_t stride = uint64_t(gridDim.x) * kThreads;
    for (uint64_t v0 = uint64_t(blockIdx.x) * kThreads + threadIdx.x; v0 < a.n; v0 += stride * kU) {
        uint4 x[kU];
#pragma unroll
        for (int u = 0; u < kU; u++) {
            const uint64_t v = v0 + uint64_t(u) * stride;
            x[u] = make_uint4(0u, 0u, 0u, 0u);
            if (v < a.n) {
                if constexpr (V == 4) x[u] = __ldcs(reinterpret_cast<const uint4 *>(a.src) + v);
                else x[u].x = __ldcs(a.src + v);
            }
        }
        for (int d = 0; d < a.n_dst; d++) {
#pragma unroll
            for (int u = 0; u < kU; u++) {
                const uint64_t v = v0 + uint64_t(u) * stride;
                if (v < a.n) {
                    if constexpr (V == 4) __stcs(reinterpret_cast<uint4 *>(a.dst[d]) + v, x[u]);
                    else __stcs(a.dst[d] + v, x[u].x);
                }
            }
        }
    }
}

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

// Bounded wait for a phase of a barrier (given by its shared-memory address); false when it gave up.  try_wait
// may keep the thread suspended in hardware for the time given as its last operand (nanoseconds), so the loop
// turns slowly and the clock is looked at every 64 turns only.
__device__ __forceinline__ bool wait_phase(uint32_t bar, uint32_t parity)
{
    long long start = 0;
    for (uint32_t turns = 0;; turns++) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
        if (ok) return true;
        if ((turns & 63u) == 63u) {
            const long long now = clock64();
            if (start == 0) start = now;
            else if (now - start > kWaitCycles) return false;
        }
    }
}

// TILE bytes per ring stage, S stages; static shared memory, so at most 48 KB together.
template <int TILE, int S>
__global__ void __launch_bounds__(32)
rd_broadcast_bulk_kernel(const __grid_constant__ BcastParams a)
{
    static_assert(TILE % 16 == 0 && S >= 2 && TILE * S + 8 * S <= 48 * 1024, "ring in static shared memory");
    __shared__ __align__(128) unsigned char ring[S][TILE];
    __shared__ __align__(8) unsigned long long full[S];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x != 0) return;
    const uint32_t ringAt = smem_addr(ring), fullAt = smem_addr(full);
#pragma unroll
    for (int s = 0; s < S; s++) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(fullAt + uint32_t(s) * 8u), "r"(1u) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");

    // tiles blockIdx.x, blockIdx.x + gridDim.x, ... of the message are this thread block's
    const uint64_t nTiles = (a.n + uint64_t(TILE) - 1) / uint64_t(TILE);
    const uint64_t mine = blockIdx.x < nTiles ? (nTiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const unsigned char *src = reinterpret_cast<const unsigned char *>(a.src);
    auto offset = [&](uint64_t k) { return (uint64_t(blockIdx.x) + k * gridDim.x) * uint64_t(TILE); };
    auto length = [&](uint64_t k) { const uint64_t left = a.n - offset(k); return uint32_t(left < uint64_t(TILE) ? left : uint64_t(TILE)); };
    auto fetch = [&](uint64_t k) {
        const uint32_t stage = uint32_t(k % S), bar = fullAt + stage * 8u, bytes = length(k);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(ringAt + stage * uint32_t(TILE)), "l"(src + offset(k)), "r"(bytes), "r"(bar) : "memory");
    };

    // the reduction that produced src has finished, and nothing reads the destinations any more
    asm volatile("griddepcontrol.wait;" ::: "memory");
    uint64_t policy;                     // the copies are not read again: first in line to leave L2
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    uint64_t fetched = 0;
    for (; fetched < mine && fetched < uint64_t(S); fetched++) fetch(fetched);
    uint64_t k = 0;
    for (; k < mine; k++) {
        const uint32_t stage = uint32_t(k % S);
        if (!wait_phase(fullAt + stage * 8u, uint32_t(k / S) & 1u)) break;
        const uint32_t bytes = length(k);
        const uint64_t at = offset(k);
        for (int d = 0; d < a.n_dst; d++)
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                         ::"l"(reinterpret_cast<unsigned char *>(a.dst[d]) + at), "r"(ringAt + stage * uint32_t(TILE)), "r"(bytes), "l"(policy) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        // the stage of the tile before this one is free once its copies have read it: fill it again
        if (k >= 1 && fetched < mine) {
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            fetch(fetched++);
        }
    }
    if (k < mine) {
        // gave up: record it, then wait (bounded again) for the copies into shared memory that are still on their way
        atomicCAS(a.status, 0, -5);
        for (uint64_t j = k; j < fetched; j++)
            if (!wait_phase(fullAt + uint32_t(j % S) * 8u, uint32_t(j / S) & 1u)) break;
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

template <typename K>
cudaError_t launch(K kernel, const BcastParams &prm, uint64_t blocks, int threads, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(blocks)); cfg.blockDim = dim3(unsigned(threads)); cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, prm);
}

cudaError_t launch_bulk(const BcastParams &prm, int sm_count, cudaStream_t stream)
{
    // thread blocks an SM holds at a time, asked once per device
    static std::atomic<int> known[kDevices];
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    int perSm = device >= 0 && device < kDevices ? known[device].load(std::memory_order_relaxed) : 0;
    if (perSm == 0) {
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&perSm, rd_broadcast_bulk_kernel<kBulkTile, kBulkStages>, 32, 0);
        if (e != cudaSuccess) return e;
        if (device >= 0 && device < kDevices) known[device].store(perSm, std::memory_order_relaxed);
    }
    const uint64_t nTiles = (prm.n + uint64_t(kBulkTile) - 1) / uint64_t(kBulkTile);
    uint64_t blocks = uint64_t(sm_count > 0 ? sm_count : 1) * uint64_t(perSm > 0 ? perSm : 1);
    if (blocks > nTiles) blocks = nTiles;
    return launch(rd_broadcast_bulk_kernel<kBulkTile, kBulkStages>, prm, blocks, 32, stream);
}

template <int V>
cudaError_t launch_registers(const BcastParams &prm, int sm_count, cudaStream_t stream)
{
    const uint64_t perBlock = uint64_t(kThreads) * kU;
    uint64_t blocks = (prm.n + perBlock - 1) / perBlock;
    const uint64_t most = uint64_t(sm_count > 0 ? sm_count : 1) * 8u;
    if (blocks > most) blocks = most;
    return launch(rd_broadcast_kernel<V>, prm, blocks, kThreads, stream);
}

}  // namespace

int broadcast_launches(int n_dst, uint64_t n_words, bool aligned)
{
    if (n_dst <= 0 || n_words == 0) return 0;
    const int groups = (n_dst + kBcastPackPtrs - 1) / kBcastPackPtrs;
    if (!aligned) return groups;
    return groups * ((n_words >= 4 ? 1 : 0) + ((n_words & 3u) ? 1 : 0));
}

int launch_broadcast(const void *src, void *const *dsts, int n_dst, uint64_t n_words, bool aligned, int sm_count, int *status,
                     void *stream)
{
    if (n_words == 0) return 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint64_t wideWords = aligned ? n_words & ~uint64_t(3) : 0;       // whole 128-bit vectors
    for (int base = 0; base < n_dst; base += kBcastPackPtrs) {
        BcastParams prm;
        const int cnt = n_dst - base < kBcastPackPtrs ? n_dst - base : kBcastPackPtrs;
        prm.n_dst = cnt; prm.status = status;
        if (wideWords > 0) {
            for (int i = 0; i < kBcastPackPtrs; i++) prm.dst[i] = i < cnt ? static_cast<uint32_t *>(dsts[base + i]) : nullptr;
            prm.src = static_cast<const uint32_t *>(src);
            prm.n = n_dst <= kBulkMostDst ? wideWords * 4 : wideWords / 4;
            if (const cudaError_t e = n_dst <= kBulkMostDst ? launch_bulk(prm, sm_count, st) : launch_registers<4>(prm, sm_count, st))
                return int(e);
        }
        if (wideWords < n_words) {
            for (int i = 0; i < kBcastPackPtrs; i++) prm.dst[i] = i < cnt ? static_cast<uint32_t *>(dsts[base + i]) + wideWords : nullptr;
            prm.src = static_cast<const uint32_t *>(src) + wideWords;
            prm.n = n_words - wideWords;
            if (const cudaError_t e = launch_registers<1>(prm, sm_count, st)) return int(e);
        }
    }
    return 0;
}

}  // namespace rd
