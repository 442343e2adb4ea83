// sm_100a kernels of the schedule-exact reduction.
//
// Tree kernel: every thread owns U vectors of V elements of the message and evaluates, for them,
// the segment's combine program: a one-accumulator stack machine whose operands are the p
// processes' elements at the same index.  The path is bound by HBM (4(p+1) bytes per output
// element, p-1 combines), so the kernel is built around keeping many independent 128-bit loads in
// flight per thread: operands are fetched K operations ahead, in program order, into a register
// ring that is statically indexed by unrolling the interpreter K times.  Partial results that have
// to wait (at most log2 p of them) live in a per-thread column of shared memory.
#include <cuda_runtime.h>

#include <cstdint>

#include "rd_kernels.h"

namespace rd {

namespace {

constexpr int kIdxBits = 12;
constexpr uint32_t kIdxMask = (1u << kIdxBits) - 1;

enum { DT_INT32 = 0, DT_FP32 = 1 };
enum { OPR_SUM = 0, OPR_MAX = 1 };

template <int V> struct Vec { uint32_t w[V]; };

template <int V> __device__ __forceinline__ Vec<V> load_stream(const uint32_t *p);
template <> __device__ __forceinline__ Vec<4> load_stream<4>(const uint32_t *p)
{
    const uint4 v = __ldcs(reinterpret_cast<const uint4 *>(p));
    Vec<4> r; r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[3] = v.w; return r;
}
template <> __device__ __forceinline__ Vec<1> load_stream<1>(const uint32_t *p)
{
    Vec<1> r; r.w[0] = __ldcs(p); return r;
}
template <int V> __device__ __forceinline__ void store_stream(uint32_t *p, const Vec<V> &v);
template <> __device__ __forceinline__ void store_stream<4>(uint32_t *p, const Vec<4> &v)
{
    __stcs(reinterpret_cast<uint4 *>(p), make_uint4(v.w[0], v.w[1], v.w[2], v.w[3]));
}
template <> __device__ __forceinline__ void store_stream<1>(uint32_t *p, const Vec<1> &v) { __stcs(p, v.w[0]); }

// combine(held, incoming): what a receiver does with the segment it holds and the one that arrives.
template <int DT, int OPR> __device__ __forceinline__ uint32_t combine(uint32_t held, uint32_t in)
{
    if (DT == DT_INT32) {
        if (OPR == OPR_SUM) return held + in;                       // wraps modulo 2^32
        return (int32_t(in) > int32_t(held)) ? in : held;
    } else {
        const float h = __uint_as_float(held), i = __uint_as_float(in);
        if (OPR == OPR_SUM) return __float_as_uint(__fadd_rn(h, i));   // one IEEE add, never contracted
        return (i > h) ? in : held;
    }
}

struct PtrPack { const uint32_t *ptr[kPackedPtrs]; };
struct PtrRef { const uint32_t *const *table; };

template <bool PACKED> struct TreeParams;
template <> struct TreeParams<true> {
    PtrPack in;
    uint32_t *out; const TileDesc *tiles; const uint32_t *ops; uint32_t n_tiles; int p;
    __device__ __forceinline__ const uint32_t *input(uint32_t i) const { return in.ptr[i]; }
};
template <> struct TreeParams<false> {
    PtrRef in;
    uint32_t *out; const TileDesc *tiles; const uint32_t *ops; uint32_t n_tiles; int p;
    __device__ __forceinline__ const uint32_t *input(uint32_t i) const { return reinterpret_cast<const uint32_t *>(__ldg(reinterpret_cast<const unsigned long long *>(in.table) + i));
    }
};

template <int DT, int OPR, int V, int U, int K, bool PACKED>
__global__ void __launch_bounds__(kTreeThreads, 2)
rd_tree_kernel(const __grid_constant__ TreeParams<PACKED> a)
{
    extern __shared__ uint4 stack_raw[];
    Vec<V> *stack = reinterpret_cast<Vec<V> *>(stack_raw);   // [depth][U][threads]
    const uint32_t tid = threadIdx.x;
    const int p = a.p;

    for (uint32_t tile = blockIdx.x; tile < a.n_tiles; tile += gridDim.x) {
        const TileDesc td = a.tiles[tile];
        const uint32_t *prog = a.ops + td.prog;
        uint32_t eoff[U];
        bool live[U];
#pragma unroll
        for (int u = 0; u < U; u++) {
            eoff[u] = (uint32_t(u) * kTreeThreads + tid) * V;
            live[u] = eoff[u] < td.len;
        }
        Vec<V> ring[K][U];
#pragma unroll
        for (int k = 0; k < K; k++) {
            if (k < p) {
                const uint32_t *src = a.input(__ldg(prog + k) & kIdxMask) + td.elem_off;
#pragma unroll
                for (int u = 0; u < U; u++)
                    if (live[u]) ring[k][u] = load_stream<V>(src + eoff[u]);
            }
        }
        Vec<V> top[U];
#pragma unroll
        for (int u = 0; u < U; u++)
#pragma unroll
            for (int v = 0; v < V; v++) top[u].w[v] = 0;
        int sp = 0;
        for (int base = 0; base < p; base += K) {
#pragma unroll
            for (int k = 0; k < K; k++) {
                const int i = base + k;
                if (i < p) {
                    const uint32_t w = __ldg(prog + i);
                    Vec<V> x[U];
#pragma unroll
                    for (int u = 0; u < U; u++) x[u] = ring[k][u];
                    if (i + K < p) {                       // refill this ring slot, K operations ahead
                        const uint32_t *src = a.input(__ldg(prog + i + K) & kIdxMask) + td.elem_off;
#pragma unroll
                        for (int u = 0; u < U; u++)
                            if (live[u]) ring[k][u] = load_stream<V>(src + eoff[u]);
                    }
                    const uint32_t kind = (w >> kIdxBits) & 3u;
                    if (kind == 1u) {                      // PUSH_LOAD
#pragma unroll
                        for (int u = 0; u < U; u++) stack[(sp * U + u) * kTreeThreads + tid] = top[u];
                        sp++;
                    }
                    if (kind <= 1u) {                      // LOAD / PUSH_LOAD
#pragma unroll
                        for (int u = 0; u < U; u++) top[u] = x[u];
                    } else if (kind == 2u || OPR == OPR_SUM) {   // ACC_IN (a sum does not care who held what)
#pragma unroll
                        for (int u = 0; u < U; u++)
#pragma unroll
                            for (int v = 0; v < V; v++) top[u].w[v] = combine<DT, OPR>(top[u].w[v], x[u].w[v]);
                    } else {                               // ACC_HELD
#pragma unroll
                        for (int u = 0; u < U; u++)
#pragma unroll
                            for (int v = 0; v < V; v++) top[u].w[v] = combine<DT, OPR>(x[u].w[v], top[u].w[v]);
                    }
                    uint32_t npop = (w >> (kIdxBits + 2)) & 0xFu;
                    uint32_t roles = w >> (kIdxBits + 6);
                    while (npop--) {
                        sp--;
                        const bool poppedHeld = (roles & 1u) != 0;
                        roles >>= 1;
#pragma unroll
                        for (int u = 0; u < U; u++) {
                            const Vec<V> y = stack[(sp * U + u) * kTreeThreads + tid];
#pragma unroll
                            for (int v = 0; v < V; v++)
                                top[u].w[v] = (poppedHeld || OPR == OPR_SUM) ? combine<DT, OPR>(y.w[v], top[u].w[v])
                                                                            : combine<DT, OPR>(top[u].w[v], y.w[v]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; u++)
            if (live[u]) store_stream<V>(a.out + td.elem_off + eoff[u], top[u]);
    }
}

constexpr int kU = 2;   // vectors per thread per operation
constexpr int kK = 4;   // operations fetched ahead

template <int DT, int OPR, int V, bool PACKED>
cudaError_t launch_one(const TreeLaunch &l)
{
    TreeParams<PACKED> prm;
    if constexpr (PACKED) {
        for (int i = 0; i < kPackedPtrs; i++) prm.in.ptr[i] = i < l.p ? static_cast<const uint32_t *>(l.host_ptrs[i]) : nullptr;
    } else {
        prm.in.table = reinterpret_cast<const uint32_t *const *>(l.dev_ptr_table);
    }
    prm.out = static_cast<uint32_t *>(l.out);
    prm.tiles = l.tiles; prm.ops = l.ops; prm.n_tiles = l.n_tiles; prm.p = l.p;
    auto kernel = rd_tree_kernel<DT, OPR, V, kU, kK, PACKED>;
    const int depth = l.stack_depth > 0 ? l.stack_depth : 1;
    const size_t smem = size_t(depth) * kU * kTreeThreads * sizeof(Vec<V>);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    int perSm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&perSm, kernel, kTreeThreads, smem);
    if (e != cudaSuccess) return e;
    if (perSm < 1) perSm = 1;
    uint32_t grid = uint32_t(l.sm_count) * uint32_t(perSm);
    if (grid > l.n_tiles) grid = l.n_tiles;
    kernel<<<grid, kTreeThreads, smem, static_cast<cudaStream_t>(l.stream)>>>(prm);
    return cudaGetLastError();
}

template <int DT, int OPR>
cudaError_t launch_dtop(const TreeLaunch &l)
{
    const bool packed = l.p <= kPackedPtrs;
    if (l.vec == 4) return packed ? launch_one<DT, OPR, 4, true>(l) : launch_one<DT, OPR, 4, false>(l);
    return packed ? launch_one<DT, OPR, 1, true>(l) : launch_one<DT, OPR, 1, false>(l);
}

}  // namespace

uint32_t tree_tile_elems(int vec) { return uint32_t(kTreeThreads) * kU * uint32_t(vec); }

int launch_tree(const TreeLaunch &l)
{
    if (l.n_tiles == 0) return 0;
    cudaError_t e;
    if (l.dtype == DT_INT32) e = l.op == OPR_SUM ? launch_dtop<DT_INT32, OPR_SUM>(l) : launch_dtop<DT_INT32, OPR_MAX>(l);
    else e = l.op == OPR_SUM ? launch_dtop<DT_FP32, OPR_SUM>(l) : launch_dtop<DT_FP32, OPR_MAX>(l);
    return int(e);
}

}  // namespace rd
