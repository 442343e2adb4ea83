// sm_100a kernels of the schedule-exact reduction, tree mode.
//
// Every thread owns a few 128-bit vectors of the message and evaluates, for them, the segment's
// combine program: a one-accumulator stack machine whose operands are the p processes' elements at
// the same index.  The path is bound by HBM (4(p+1) bytes per output element, p-1 combines), so the
// kernels are built around keeping many bytes in flight:
//   rd_tree_stream_kernel  the throughput path (128-bit aligned buffers): operand tiles are streamed
//                          into a shared-memory ring by bulk asynchronous copies issued by producer
//                          threads, consumers execute the program on them;
//   rd_tree_direct_kernel  few processes, on request: all operands of an element in registers at once;
//   rd_tree_kernel         the element path (buffers aligned to the element only): operands are fetched K
//                          operations ahead, in program order, into a register ring that is
//                          statically indexed by unrolling the interpreter K times.
// Partial results that have to wait (at most log2 p of them) live in a per-thread column of shared
// memory in both.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <map>
#include <mutex>

#include "rd_kernels.h"

namespace rd {

namespace {

// Dynamic shared memory: every kernel instantiation that uses it is opted into the device's largest
// per-block size exactly once per device, under a lock, before its first launch there.  The limit then
// never moves again, so launches of different ring shapes from different threads cannot undercut each
// other (setting it per launch to that launch's own size could leave it below what a concurrent launch
// of a larger shape was about to ask for).
inline cudaError_t opt_in_shared_memory(const void *kernel, int device)
{
    static std::mutex lock;
    static std::map<const void *, uint64_t> done;            // kernel -> devices it has been opted in on
    if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> hold(lock);
    uint64_t &mask = done[kernel];
    if (mask >> device & 1u) return cudaSuccess;
    int most = 0;
    cudaError_t e = cudaDeviceGetAttribute(&most, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, kernel);                  // the limit covers static and dynamic shared memory together
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, most - int(fa.sharedSizeBytes));
    if (e != cudaSuccess) return e;
    mask |= uint64_t(1) << device;
    return cudaSuccess;
}

constexpr int kIdxBits = 12;
constexpr uint32_t kIdxMask = (1u << kIdxBits) - 1;

// DT_BF16_PICK, DT_FP16_PICK: the 16-bit types under max and min.  The result of such a combine is one of its
// two operands, so nothing ever leaves the 16-bit format: the kernels work on the packed pairs of a word
// directly (one packed comparison and one bit select per word), partial results are as large as the
// operands, and the result equals, bit for bit, that of widening to fp32, comparing there and rounding at
// the end (widening keeps the order, the selected value is representable).
enum { DT_INT32 = 0, DT_FP32 = 1, DT_INT64 = 2, DT_FP64 = 3, DT_BF16 = 4, DT_FP16 = 5, DT_BF16_PICK = 6, DT_FP16_PICK = 7 };

// The kernels move and index the message in 32-bit words; an element is one word or two, or (bf16, fp16)
// half a word: a word then holds two elements, the lower-addressed one in its low half.
template <int DT> struct ElemWords { static constexpr int value = (DT == DT_INT64 || DT == DT_FP64) ? 2 : 1; };
// 16-bit elements are combined in fp32: a word of the message becomes W = 2 words of partial result (two
// fp32 values), the arithmetic is that of fp32, and only the root's value is rounded back to 16 bits.
template <int DT> struct Wide {
    static constexpr bool half = DT == DT_BF16 || DT == DT_FP16;
    static constexpr int W = half ? 2 : 1;
    static constexpr int ADT = half ? DT_FP32 : DT;
};
enum { OPR_SUM = 0, OPR_MAX = 1, OPR_MIN = 2, OPR_PROD = 3 };
enum { LAUNCH_STREAM = 0, LAUNCH_BATCH = 1, LAUNCH_DIRECT = 2, LAUNCH_ELEMENT = 3 };

template <int V> struct Vec { uint32_t w[V]; };

template <int V> __device__ __forceinline__ Vec<V> load_stream(const uint32_t *p);
template <> __device__ __forceinline__ Vec<1> load_stream<1>(const uint32_t *p)
{
    Vec<1> r; r.w[0] = __ldcs(p); return r;
}
template <> __device__ __forceinline__ Vec<2> load_stream<2>(const uint32_t *p)
{
    const uint2 t = __ldcs(reinterpret_cast<const uint2 *>(p));
    Vec<2> r; r.w[0] = t.x; r.w[1] = t.y; return r;
}
template <int V> __device__ __forceinline__ void store_stream(uint32_t *p, const Vec<V> &v);
template <> __device__ __forceinline__ void store_stream<2>(uint32_t *p, const Vec<2> &v)
{
    __stcs(reinterpret_cast<uint2 *>(p), make_uint2(v.w[0], v.w[1]));
}
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
        if (OPR == OPR_PROD) return held * in;                      // wraps modulo 2^32
        if (OPR == OPR_MAX) return (int32_t(in) > int32_t(held)) ? in : held;
        return (int32_t(in) < int32_t(held)) ? in : held;
    } else if (DT == DT_BF16_PICK || DT == DT_FP16_PICK) {
        // two elements per word: all ones in the half where the incoming element wins (never on a tie or a NaN)
        unsigned wins;
        if (DT == DT_BF16_PICK) {
            const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162 *>(&held), i = *reinterpret_cast<const __nv_bfloat162 *>(&in);
            wins = OPR == OPR_MAX ? __hgt2_mask(i, h) : __hlt2_mask(i, h);
        } else {
            const __half2 h = *reinterpret_cast<const __half2 *>(&held), i = *reinterpret_cast<const __half2 *>(&in);
            wins = OPR == OPR_MAX ? __hgt2_mask(i, h) : __hlt2_mask(i, h);
        }
        return (in & wins) | (held & ~wins);
    } else {
        const float h = __uint_as_float(held), i = __uint_as_float(in);
        if (OPR == OPR_SUM) return __float_as_uint(__fadd_rn(h, i));   // one IEEE add, never contracted
        if (OPR == OPR_PROD) return __float_as_uint(__fmul_rn(h, i));  // one IEEE multiply
        if (OPR == OPR_MAX) return (i > h) ? in : held;
        return (i < h) ? in : held;
    }
}

// The same for the 8-byte element types (low word first in memory).
template <int DT, int OPR> __device__ __forceinline__ unsigned long long combine64(unsigned long long held, unsigned long long in)
{
    if (DT == DT_INT64) {
        if (OPR == OPR_SUM) return held + in;                       // wraps modulo 2^64
        if (OPR == OPR_PROD) return held * in;                      // wraps modulo 2^64
        if (OPR == OPR_MAX) return ((long long)in > (long long)held) ? in : held;
        return ((long long)in < (long long)held) ? in : held;
    } else {
        const double h = __longlong_as_double((long long)held), i = __longlong_as_double((long long)in);
        if (OPR == OPR_SUM) return (unsigned long long)__double_as_longlong(__dadd_rn(h, i));
        if (OPR == OPR_PROD) return (unsigned long long)__double_as_longlong(__dmul_rn(h, i));
        if (OPR == OPR_MAX) return (i > h) ? in : held;
        return (i < h) ? in : held;
    }
}

// Two fp32 sums (products) in one instruction: sm_100's packed single-precision add (multiply) works on a pair of
// registers, each half one IEEE operation rounded to nearest even like the scalar one, subnormals kept.
template <int OPR> __device__ __forceinline__ void combine_pair_f32(uint32_t &r0, uint32_t &r1, uint32_t h0, uint32_t h1, uint32_t i0, uint32_t i1)
{
    if (OPR == OPR_SUM)
        asm("{\n\t.reg .b64 a, b, c;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 b, {%4, %5};\n\tadd.rn.f32x2 c, a, b;\n\tmov.b64 {%0, %1}, c;\n\t}"
            : "=r"(r0), "=r"(r1) : "r"(h0), "r"(h1), "r"(i0), "r"(i1));
    else
        asm("{\n\t.reg .b64 a, b, c;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 b, {%4, %5};\n\tmul.rn.f32x2 c, a, b;\n\tmov.b64 {%0, %1}, c;\n\t}"
            : "=r"(r0), "=r"(r1) : "r"(h0), "r"(h1), "r"(i0), "r"(i1));
}

// A vector of V words: V elements of a 4-byte type, V / 2 of an 8-byte type.  r may be held or in.
template <int DT, int OPR, int V> __device__ __forceinline__ void combine_vec(Vec<V> &r, const Vec<V> &held, const Vec<V> &in)
{
    if constexpr (DT == DT_FP32 && (OPR == OPR_SUM || OPR == OPR_PROD) && V % 2 == 0) {
#pragma unroll
        for (int v = 0; v < V; v += 2) combine_pair_f32<OPR>(r.w[v], r.w[v + 1], held.w[v], held.w[v + 1], in.w[v], in.w[v + 1]);
    } else if constexpr (ElemWords<DT>::value == 1) {
#pragma unroll
        for (int v = 0; v < V; v++) r.w[v] = combine<DT, OPR>(held.w[v], in.w[v]);
    } else {
        static_assert(V % 2 == 0, "an 8-byte element never straddles two vectors");
#pragma unroll
        for (int v = 0; v < V; v += 2) {
            const unsigned long long h = (unsigned long long)held.w[v] | ((unsigned long long)held.w[v + 1] << 32);
            const unsigned long long i = (unsigned long long)in.w[v] | ((unsigned long long)in.w[v + 1] << 32);
            const unsigned long long c = combine64<DT, OPR>(h, i);
            r.w[v] = uint32_t(c); r.w[v + 1] = uint32_t(c >> 32);
        }
    }
}

// A vector of V message words as V * W words of partial result, and back (bf16, fp16: exact widening, one
// rounding to nearest even on the way back; other types: the same words).
template <int DT, int V> __device__ __forceinline__ Vec<V * Wide<DT>::W> widen(const Vec<V> &m)
{
    Vec<V * Wide<DT>::W> a;
    if constexpr (Wide<DT>::W == 1) {
#pragma unroll
        for (int v = 0; v < V; v++) a.w[v] = m.w[v];
    } else {
#pragma unroll
        for (int v = 0; v < V; v++) {
            if constexpr (DT == DT_BF16) {                      // a bf16 is the upper half of an fp32
                a.w[2 * v] = m.w[v] << 16; a.w[2 * v + 1] = m.w[v] & 0xFFFF0000u;
            } else {
                a.w[2 * v] = __float_as_uint(__half2float(__ushort_as_half((unsigned short)(m.w[v] & 0xFFFFu))));
                a.w[2 * v + 1] = __float_as_uint(__half2float(__ushort_as_half((unsigned short)(m.w[v] >> 16))));
            }
        }
    }
    return a;
}
template <int DT, int V> __device__ __forceinline__ Vec<V> narrow(const Vec<V * Wide<DT>::W> &a)
{
    Vec<V> m;
    if constexpr (Wide<DT>::W == 1) {
#pragma unroll
        for (int v = 0; v < V; v++) m.w[v] = a.w[v];
    } else {
#pragma unroll
        for (int v = 0; v < V; v++) {
            uint32_t lo, hi;
            if constexpr (DT == DT_BF16) {
                lo = __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(a.w[2 * v])));
                hi = __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(a.w[2 * v + 1])));
            } else {
                lo = __half_as_ushort(__float2half_rn(__uint_as_float(a.w[2 * v])));
                hi = __half_as_ushort(__float2half_rn(__uint_as_float(a.w[2 * v + 1])));
            }
            m.w[v] = lo | (hi << 16);
        }
    }
    return m;
}

// Sum and product give the same bits whichever operand was held (IEEE add and multiply commute), and so do max and
// min of integers (equal integers are the same bits; floating-point zeros of either sign compare equal, so there the
// held operand has to be known).
template <int DT, int OPR> struct Commutes {
    static constexpr bool value = OPR == OPR_SUM || OPR == OPR_PROD || DT == DT_INT32 || DT == DT_INT64;
};

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
    constexpr int AV = V * Wide<DT>::W;                       // words of partial result per vector
    constexpr int ADT = Wide<DT>::ADT;
    extern __shared__ uint4 stack_raw[];
    Vec<AV> *stack = reinterpret_cast<Vec<AV> *>(stack_raw);  // [depth][U][threads]
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
        Vec<AV> top[U];
#pragma unroll
        for (int u = 0; u < U; u++)
#pragma unroll
            for (int v = 0; v < AV; v++) top[u].w[v] = 0;
        int sp = 0;
        for (int base = 0; base < p; base += K) {
#pragma unroll
            for (int k = 0; k < K; k++) {
                const int i = base + k;
                if (i < p) {
                    const uint32_t w = __ldg(prog + i);
                    Vec<AV> x[U];
#pragma unroll
                    for (int u = 0; u < U; u++) x[u] = widen<DT, V>(ring[k][u]);
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
                    } else if (kind == 2u || Commutes<DT, OPR>::value) {   // ACC_IN (a sum does not care who held what)
#pragma unroll
                        for (int u = 0; u < U; u++) combine_vec<ADT, OPR, AV>(top[u], top[u], x[u]);
                    } else {                               // ACC_HELD
#pragma unroll
                        for (int u = 0; u < U; u++) combine_vec<ADT, OPR, AV>(top[u], x[u], top[u]);
                    }
                    uint32_t npop = (w >> (kIdxBits + 2)) & 0xFu;
                    uint32_t roles = w >> (kIdxBits + 6);
                    while (npop--) {
                        sp--;
                        const bool poppedHeld = (roles & 1u) != 0;
                        roles >>= 1;
#pragma unroll
                        for (int u = 0; u < U; u++) {
                            const Vec<AV> y = stack[(sp * U + u) * kTreeThreads + tid];
                            if (poppedHeld || Commutes<DT, OPR>::value) combine_vec<ADT, OPR, AV>(top[u], y, top[u]);
                            else combine_vec<ADT, OPR, AV>(top[u], top[u], y);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; u++)
            if (live[u]) store_stream<V>(a.out + td.elem_off + eoff[u], narrow<DT, V>(top[u]));
    }
}

// ---------------------------------------------------------------------------------------------
// Streaming variant (128-bit path).  Two producer threads per CTA (one per producer warp) walk the
// CTA's (tile, operation) pairs in program order and issue one bulk asynchronous copy
// (cp.async.bulk, global -> shared, completion counted in bytes on an mbarrier) per operand tile
// into a ring of 8 KB shared-memory stages; they run ahead across tile boundaries, so the number of
// bytes in flight per SM is set by the ring, not by registers or scoreboards.  The consumer warps
// (8 or 4) take the stages in the same order, each thread reading its vectors of the stage, and
// execute the program on them.  A stage holds one operand tile of up to 2048 words, or two of up to
// 1024 (see StreamShape).
// Every wait is bounded: on expiry the thread records an error code and the CTA winds down (a
// producer lane first waits, again bounded, for the copy it has in flight).
// ---------------------------------------------------------------------------------------------
constexpr int kStageWords = 2048;                       // a ring stage: 8 KB; the largest tile
constexpr int kStageVecs = kStageWords / 4;
constexpr int kMaxStages = 32;
constexpr int kProducers = 2;                            // producer warps per CTA (one active lane each)
constexpr long long kWaitCycles = 4000000000ll;         // a wait gives up after about two seconds of SM clock

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

// Waits on a barrier given by its shared-memory address.  The last operand is a hint: the thread may stay
// suspended in hardware up to that many nanoseconds while the phase is not complete (it resumes when it is), so
// a waiting thread spends few issue slots.
__device__ __forceinline__ bool mbar_try_wait_at(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
    return ok != 0;
}
// Bounded wait; false when it gave up or another thread of the CTA already did.  try_wait suspends
// the thread in hardware for a while, so the loop turns slowly; the clock and the abort flag are
// only looked at every 64 turns.
__device__ __forceinline__ bool mbar_wait_at(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait_at(bar, parity)) return true;
    long long start = 0;
    for (uint32_t turns = 1;; turns++) {
        if (mbar_try_wait_at(bar, parity)) return true;
        if ((turns & 63u) == 0u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (start == 0) start = now;
            else if (now - start > kWaitCycles) return false;
        }
    }
}
__device__ __forceinline__ void mbar_arrive_at(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr) : "memory");
    return r;
}
__device__ __forceinline__ void sts128(uint32_t addr, const uint4 &v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void bulk_load_at(uint32_t smem_dst, const void *gmem_src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_at(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

constexpr uint32_t kLenMask = 0xFFFFu;   // TileDesc::len: bits 0-15 padded length, 16-17 elements to skip at the head, 18-19 at the tail

// Stores a 4-element vector, or only elements [skip_head, 4 - skip_tail) of it.
__device__ __forceinline__ void store_part(uint32_t *p, const Vec<4> &v, uint32_t skip_head, uint32_t skip_tail)
{
    if ((skip_head | skip_tail) == 0u) { store_stream<4>(p, v); return; }
#pragma unroll
    for (uint32_t e = 0; e < 4u; e++)
        if (e >= skip_head && e < 4u - skip_tail) __stcs(p + e, v.w[e]);
}

// What a launch works on is reached through a "jobs" view: one reduction (the view is the kernel's
// parameters and costs nothing), or several independent reductions fused into one launch (the tiles
// of all jobs are numbered through; the view keeps the descriptor of the job its tile belongs to).
template <bool PACKED> struct OneJob;
template <bool PACKED> struct ManyJobs;

template <bool PACKED> struct StreamParams {
    using Jobs = OneJob<PACKED>;
    TreeParams<PACKED> t;
    const uint32_t *cta_first;   // per CTA: first tile; n_ctas + 1 entries
    int *status;                 // device word: 0, or the first error code
    uint32_t *tile_counter;      // two device words (next tile, CTAs done), both 0 at launch: tiles are handed out
                                 // on demand; null: every CTA works through its own range
    int stages, depth;
    __device__ __forceinline__ void tile_range(uint32_t cta, uint32_t &t0, uint32_t &t1) const { t0 = cta_first[cta]; t1 = cta_first[cta + 1]; }
    __device__ __forceinline__ uint32_t total_tiles() const { return t.n_tiles; }
};

// A batch: job descriptors and input pointers either inside the kernel's parameters (small batches: nothing
// has to be copied to the device before the launch) or in device memory.  CTA c of n takes the tiles
// [T c / n, T (c + 1) / n) of the batch's T tiles.
template <bool PACKED> struct BatchStreamParams;
template <> struct BatchStreamParams<true> {
    using Jobs = ManyJobs<true>;
    BatchJob jobs[kBatchPackJobs];
    const uint32_t *ptrs[kBatchPackPtrs];
    uint32_t n_jobs, n_tiles;
    int *status;
    uint32_t *tile_counter;
    int stages, depth;
    __device__ __forceinline__ uint32_t total_tiles() const { return n_tiles; }
    __device__ __forceinline__ BatchJob job(uint32_t j) const { return jobs[j]; }
    __device__ __forceinline__ uint32_t job_end(uint32_t j) const { return jobs[j].tile_end; }
    __device__ __forceinline__ const uint32_t *input(const BatchJob &b, uint32_t i) const { return ptrs[uint32_t(b.ptr_base) + i]; }
    __device__ __forceinline__ void tile_range(uint32_t cta, uint32_t &t0, uint32_t &t1) const
    {
        t0 = uint32_t(uint64_t(n_tiles) * cta / gridDim.x); t1 = uint32_t(uint64_t(n_tiles) * (cta + 1u) / gridDim.x);
    }
};
template <> struct BatchStreamParams<false> {
    using Jobs = ManyJobs<false>;
    const BatchJob *jobs;        // device; n_jobs descriptors, tile ranges ascending
    uint32_t n_jobs, n_tiles;
    int *status;
    uint32_t *tile_counter;
    int stages, depth;
    __device__ __forceinline__ uint32_t total_tiles() const { return n_tiles; }
    __device__ __forceinline__ BatchJob job(uint32_t j) const { return jobs[j]; }
    __device__ __forceinline__ uint32_t job_end(uint32_t j) const { return jobs[j].tile_end; }
    __device__ __forceinline__ const uint32_t *input(const BatchJob &b, uint32_t i) const
    {
        return reinterpret_cast<const uint32_t *>(__ldg(reinterpret_cast<const unsigned long long *>(b.inputs) + i));
    }
    __device__ __forceinline__ void tile_range(uint32_t cta, uint32_t &t0, uint32_t &t1) const
    {
        t0 = uint32_t(uint64_t(n_tiles) * cta / gridDim.x); t1 = uint32_t(uint64_t(n_tiles) * (cta + 1u) / gridDim.x);
    }
};

template <bool PACKED> struct OneJob {
    const TreeParams<PACKED> &t;
    __device__ __forceinline__ OneJob(const StreamParams<PACKED> &a, uint32_t, bool) : t(a.t) {}
    __device__ __forceinline__ void seek(uint32_t) {}
    __device__ __forceinline__ TileDesc tile(uint32_t g) const { return t.tiles[g]; }
    __device__ __forceinline__ const uint32_t *ops() const { return t.ops; }
    __device__ __forceinline__ const uint32_t *input(uint32_t i) const { return t.input(i); }
    __device__ __forceinline__ uint32_t *out() const { return t.out; }
    __device__ __forceinline__ int p() const { return t.p; }
};

template <bool PACKED> struct ManyJobs {
    const BatchStreamParams<PACKED> &a;
    BatchJob cur;
    uint32_t j;
    // Positioned on the job of tile g (the first job whose range ends after g) when `any` is set.
    __device__ __forceinline__ ManyJobs(const BatchStreamParams<PACKED> &prm, uint32_t g, bool any) : a(prm), j(0)
    {
        cur = BatchJob{nullptr, nullptr, nullptr, nullptr, 0u, 0u, 1, 0};
        if (!any) return;
        uint32_t lo = 0, hi = a.n_jobs - 1u;
        while (lo < hi) {
            const uint32_t mid = (lo + hi) / 2u;
            if (g >= a.job_end(mid)) lo = mid + 1u; else hi = mid;
        }
        j = lo;
        cur = a.job(j);
    }
    // Tiles are visited in ascending order, so the job only ever moves forward.
    __device__ __forceinline__ void seek(uint32_t g) { while (g >= cur.tile_end) cur = a.job(++j); }
    __device__ __forceinline__ TileDesc tile(uint32_t g) const { return cur.tiles[g - cur.tile_begin]; }
    __device__ __forceinline__ const uint32_t *ops() const { return cur.ops; }
    __device__ __forceinline__ const uint32_t *input(uint32_t i) const { return a.input(cur, i); }
    __device__ __forceinline__ uint32_t *out() const { return cur.out; }
    __device__ __forceinline__ int p() const { return cur.p; }
};

// ---- which tiles a CTA works on.  One producer thread decides (from the CTA's own range, or by taking
// the next tile from a counter all CTAs of the launch share, so that CTAs which get through their tiles
// faster take more of them) and publishes the sequence through a small queue in shared memory; the other
// producer and the consumers read it.  An entry is written long before it is needed and overwritten only
// kTileQ tiles later, when every reader is past it (nobody is more than a ring of stages, i.e. at most
// kMaxStages tiles, behind the writer).
constexpr uint32_t kNoTile = 0xFFFFFFFFu;
constexpr uint32_t kTileQ = 64;
static_assert(kTileQ > uint32_t(kMaxStages) + 2u, "a queue entry must outlive the ring's look-ahead");

struct TileQueue {
    uint32_t slot[kTileQ];
    uint32_t published;          // entries written so far
};

// Reader side: the k-th tile of this CTA, kNoTile after the last one.  Bounded wait; when it gives up (or
// another thread of the CTA already did) the CTA winds down: kNoTile, with the error recorded.
__device__ __forceinline__ uint32_t tile_at(TileQueue *q, uint32_t k, volatile int *abort_flag, int *status)
{
    volatile uint32_t *pub = &q->published;
    if (*pub <= k) {
        const long long start = clock64();
        while (*pub <= k) {
            if (*abort_flag) return kNoTile;
            if (clock64() - start > kWaitCycles) {
                atomicCAS(status, 0, -5);
                *abort_flag = 1;
                return kNoTile;
            }
        }
    }
    __threadfence_block();
    return reinterpret_cast<volatile uint32_t *>(q->slot)[k % kTileQ];
}

// Writer side (one thread per CTA).  With a shared counter, CTA c starts with tile c and the counter hands
// out the tiles from the number of CTAs on; the id of the next entry is fetched while the current tile is
// being issued, so that the counter's round trip to L2 is over when the entry is published.
struct TileSource {
    TileQueue *q;
    uint32_t *counter;           // null: the CTA's own range [next, end)
    uint32_t next, end, total, base;
    uint32_t pub;                // entries published
    uint32_t ahead;              // id fetched for the next entry
    bool drained;                // the source has returned kNoTile (it is asked no more after that)
    __device__ __forceinline__ uint32_t fetch()
    {
        if (drained) return kNoTile;
        uint32_t t;
        if (counter) { t = atomicAdd(counter, 1u) + base; if (t >= total) t = kNoTile; }
        else { t = next < end ? next++ : kNoTile; }
        if (t == kNoTile) drained = true;
        return t;
    }
    __device__ __forceinline__ void start(TileQueue *queue, uint32_t *ctr, uint32_t t0, uint32_t t1, uint32_t n)
    {
        q = queue; counter = ctr; next = t0; end = t1; total = n; base = gridDim.x; pub = 0; drained = false;
        if (counter) ahead = blockIdx.x < total ? blockIdx.x : kNoTile;
        else ahead = fetch();
        if (ahead == kNoTile) drained = true;
    }
    __device__ __forceinline__ void publish_one()
    {
        reinterpret_cast<volatile uint32_t *>(q->slot)[pub % kTileQ] = ahead;
        __threadfence_block();
        *reinterpret_cast<volatile uint32_t *>(&q->published) = ++pub;
        ahead = fetch();
    }
    // the k-th tile (publishing it if it is not out yet; the fetch for entry k + 1 is then under way)
    __device__ __forceinline__ uint32_t get(uint32_t k)
    {
        while (pub <= k) publish_one();
        return reinterpret_cast<volatile uint32_t *>(q->slot)[k % kTileQ];
    }
    // called after a step of tile k has been issued: entry k + 1 goes out ahead of need
    __device__ __forceinline__ void poke(uint32_t k)
    {
        if (pub == k + 1u) publish_one();
    }
    // After the last tile: the CTA that is last to run dry puts the two words back to 0 for the next launch
    // that is given them.
    __device__ __forceinline__ void finish(uint32_t n_ctas)
    {
        if (!counter) return;
        while (!drained) (void)fetch();          // (a CTA that stopped early still takes its end marker)
        __threadfence();
        if (atomicAdd(counter + 1, 1u) == n_ctas - 1u) {
            counter[0] = 0u; counter[1] = 0u;
            __threadfence();
        }
    }
};

// ---- arithmetic of the streaming kernel's accumulators.
// A consumer thread's running value lives in registers for the whole life of the thread, across the branches of the
// interpreter.  Written as ordinary assignments, every branch that leaves it alone (or changes it) ends in a block of
// register-to-register copies that bring "the new value" to the place the join expects (a third of all executed
// instructions were such copies).  So every write to an accumulator is one instruction whose destination is tied to
// the accumulator's own register (an asm operand that is input and output at once): the value never changes place.
//   acc_word<ADT, OPR, HELD>(t, x)          t = combine(t, x) (HELD: t is the held operand) or combine(x, t); one word
//   acc_pair<ADT, OPR, HELD>(t0, t1, x0, x1)  the same for two words: one 8-byte element, or two fp32 values under sum
//                                           and product (sm_100's packed add and multiply: two IEEE operations, each
//                                           rounded to nearest even like the scalar one, subnormals kept)
__device__ __forceinline__ void set_word(uint32_t &t, uint32_t x) { asm("mov.b32 %0, %1;" : "+r"(t) : "r"(x)); }

template <int ADT, int OPR, bool HELD> __device__ __forceinline__ void acc_word(uint32_t &t, uint32_t x)
{
    if constexpr (ADT == DT_INT32) {
        if (OPR == OPR_SUM) asm("add.s32 %0, %0, %1;" : "+r"(t) : "r"(x));                  // wraps modulo 2^32
        else if (OPR == OPR_PROD) asm("mul.lo.s32 %0, %0, %1;" : "+r"(t) : "r"(x));
        else if (OPR == OPR_MAX) asm("max.s32 %0, %0, %1;" : "+r"(t) : "r"(x));
        else asm("min.s32 %0, %0, %1;" : "+r"(t) : "r"(x));
    } else if constexpr (ADT == DT_BF16_PICK || ADT == DT_FP16_PICK) {
        // two 16-bit elements per word; `wins`: all ones in the half where the incoming element wins (never on a tie)
        const uint32_t held = HELD ? t : x, in = HELD ? x : t;
        unsigned wins;
        if (ADT == DT_BF16_PICK) {
            const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162 *>(&held), i = *reinterpret_cast<const __nv_bfloat162 *>(&in);
            wins = OPR == OPR_MAX ? __hgt2_mask(i, h) : __hlt2_mask(i, h);
        } else {
            const __half2 h = *reinterpret_cast<const __half2 *>(&held), i = *reinterpret_cast<const __half2 *>(&in);
            wins = OPR == OPR_MAX ? __hgt2_mask(i, h) : __hlt2_mask(i, h);
        }
        // t = wins ? in : held, bit by bit (lop3 0xCA: a ? b : c)
        if (HELD) asm("lop3.b32 %0, %1, %2, %0, 0xCA;" : "+r"(t) : "r"(wins), "r"(x));
        else asm("lop3.b32 %0, %1, %0, %2, 0xCA;" : "+r"(t) : "r"(wins), "r"(x));
    } else {
        static_assert(ADT == DT_FP32, "a 4-byte type");
        if (OPR == OPR_SUM) asm("add.rn.f32 %0, %0, %1;" : "+r"(t) : "r"(x));               // one IEEE add, never contracted
        else if (OPR == OPR_PROD) asm("mul.rn.f32 %0, %0, %1;" : "+r"(t) : "r"(x));
        else if (HELD) {                                                                    // (x > t) ? x : t   (min: <)
            if (OPR == OPR_MAX) asm("{\n\t.reg .pred p;\n\tsetp.gt.f32 p, %1, %0;\n\tselp.b32 %0, %1, %0, p;\n\t}" : "+r"(t) : "r"(x));
            else asm("{\n\t.reg .pred p;\n\tsetp.lt.f32 p, %1, %0;\n\tselp.b32 %0, %1, %0, p;\n\t}" : "+r"(t) : "r"(x));
        } else {                                                                            // (t > x) ? t : x
            if (OPR == OPR_MAX) asm("{\n\t.reg .pred p;\n\tsetp.gt.f32 p, %0, %1;\n\tselp.b32 %0, %0, %1, p;\n\t}" : "+r"(t) : "r"(x));
            else asm("{\n\t.reg .pred p;\n\tsetp.lt.f32 p, %0, %1;\n\tselp.b32 %0, %0, %1, p;\n\t}" : "+r"(t) : "r"(x));
        }
    }
}

#define RD_PAIR_ASM(body) asm("{\n\t.reg .b64 a, b;\n\t.reg .pred p;\n\tmov.b64 a, {%0, %1};\n\tmov.b64 b, {%2, %3};\n\t" body "\n\tmov.b64 {%0, %1}, a;\n\t}" \
                              : "+r"(t0), "+r"(t1) : "r"(x0), "r"(x1))
#define RD_PAIR_ASM_F64(body) asm("{\n\t.reg .f64 a, b;\n\t.reg .pred p;\n\tmov.b64 a, {%0, %1};\n\tmov.b64 b, {%2, %3};\n\t" body "\n\tmov.b64 {%0, %1}, a;\n\t}" \
                                  : "+r"(t0), "+r"(t1) : "r"(x0), "r"(x1))
template <int ADT, int OPR, bool HELD>
__device__ __forceinline__ void acc_pair(uint32_t &t0, uint32_t &t1, uint32_t x0, uint32_t x1)
{
    if constexpr (ADT == DT_FP32) {
        static_assert(OPR == OPR_SUM || OPR == OPR_PROD, "packed single precision: add and multiply");
        if (OPR == OPR_SUM) RD_PAIR_ASM("add.rn.f32x2 a, a, b;");
        else RD_PAIR_ASM("mul.rn.f32x2 a, a, b;");
    } else if constexpr (ADT == DT_INT64) {                    // low word first
        if (OPR == OPR_SUM) RD_PAIR_ASM("add.s64 a, a, b;");                              // wraps modulo 2^64
        else if (OPR == OPR_PROD) RD_PAIR_ASM("mul.lo.s64 a, a, b;");
        else if (OPR == OPR_MAX) RD_PAIR_ASM("max.s64 a, a, b;");
        else RD_PAIR_ASM("min.s64 a, a, b;");
    } else {
        static_assert(ADT == DT_FP64, "an 8-byte type");
        if (OPR == OPR_SUM) RD_PAIR_ASM_F64("add.rn.f64 a, a, b;");
        else if (OPR == OPR_PROD) RD_PAIR_ASM_F64("mul.rn.f64 a, a, b;");
        else if (HELD) {                                                                    // (x > t) ? x : t   (min: <)
            if (OPR == OPR_MAX) RD_PAIR_ASM_F64("setp.gt.f64 p, b, a;\n\tselp.f64 a, b, a, p;");
            else RD_PAIR_ASM_F64("setp.lt.f64 p, b, a;\n\tselp.f64 a, b, a, p;");
        } else {                                                                            // (t > x) ? t : x
            if (OPR == OPR_MAX) RD_PAIR_ASM_F64("setp.gt.f64 p, a, b;\n\tselp.f64 a, a, b, p;");
            else RD_PAIR_ASM_F64("setp.lt.f64 p, a, b;\n\tselp.f64 a, a, b, p;");
        }
    }
}
#undef RD_PAIR_ASM
#undef RD_PAIR_ASM_F64

// What a consumer thread carries for its N 128-bit vectors of an operand tile: the vectors themselves, or
// (bf16, fp16) their elements widened to fp32, twice as many words.  Created once per thread (zero), then only
// written through the tied-operand instructions above.
template <int DT, int N> struct StageAcc {
    static constexpr int W = Wide<DT>::W;
    static constexpr int ADT = Wide<DT>::ADT;
    Vec<4> v[N * W];
    __device__ __forceinline__ void clear()
    {
#pragma unroll
        for (int k = 0; k < N * W; k++)
#pragma unroll
            for (int e = 0; e < 4; e++) v[k].w[e] = 0;
    }
    // *this = the operand whose vectors are r
    __device__ __forceinline__ void load(const uint4 (&r)[N])
    {
#pragma unroll
        for (int n = 0; n < N; n++) {
            const Vec<4> m = {{r[n].x, r[n].y, r[n].z, r[n].w}};
            const Vec<4 * W> a = widen<DT, 4>(m);
#pragma unroll
            for (int k = 0; k < W; k++)
#pragma unroll
                for (int e = 0; e < 4; e++) set_word(v[n * W + k].w[e], a.w[4 * k + e]);
        }
    }
    // one 128-bit vector of operand words: *this[k] = combine(*this[k], x) (HELD) or combine(x, *this[k])
    template <int OPR, bool HELD> __device__ __forceinline__ void accumulate_vec(int k, const Vec<4> &x)
    {
        if constexpr (ElemWords<ADT>::value == 2 || (ADT == DT_FP32 && (OPR == OPR_SUM || OPR == OPR_PROD))) {
#pragma unroll
            for (int e = 0; e < 4; e += 2) acc_pair<ADT, OPR, HELD>(v[k].w[e], v[k].w[e + 1], x.w[e], x.w[e + 1]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; e++) acc_word<ADT, OPR, HELD>(v[k].w[e], x.w[e]);
        }
    }
    // *this = combine(*this, operand) (HELD: *this is the held one) or combine(operand, *this); the operand as it
    // comes from the ring, or another accumulator
    template <int OPR, bool HELD> __device__ __forceinline__ void accumulate(const uint4 (&r)[N])
    {
#pragma unroll
        for (int n = 0; n < N; n++) {
            const Vec<4> m = {{r[n].x, r[n].y, r[n].z, r[n].w}};
            const Vec<4 * W> a = widen<DT, 4>(m);
#pragma unroll
            for (int k = 0; k < W; k++) {
                const Vec<4> x = {{a.w[4 * k], a.w[4 * k + 1], a.w[4 * k + 2], a.w[4 * k + 3]}};
                accumulate_vec<OPR, HELD>(n * W + k, x);
            }
        }
    }
    template <int OPR, bool HELD> __device__ __forceinline__ void accumulate(const StageAcc &in)
    {
#pragma unroll
        for (int k = 0; k < N * W; k++) accumulate_vec<OPR, HELD>(k, in.v[k]);
    }
    // one stack level (shared-memory address): [vector][consumer thread]
    __device__ __forceinline__ void push(uint32_t level, uint32_t tid, uint32_t threads) const
    {
#pragma unroll
        for (int k = 0; k < N * W; k++) sts128(level + (uint32_t(k) * threads + tid) * 16u, make_uint4(v[k].w[0], v[k].w[1], v[k].w[2], v[k].w[3]));
    }
    // *this = combine(popped, *this) (POPPED_HELD) or combine(*this, popped), the popped value read from a stack level
    template <int OPR, bool POPPED_HELD> __device__ __forceinline__ void pop_accumulate(uint32_t level, uint32_t tid, uint32_t threads)
    {
#pragma unroll
        for (int k = 0; k < N * W; k++) {
            const uint4 y = lds128(level + (uint32_t(k) * threads + tid) * 16u);
            const Vec<4> x = {{y.x, y.y, y.z, y.w}};
            accumulate_vec<OPR, !POPPED_HELD>(k, x);
        }
    }
    __device__ __forceinline__ void result(Vec<4> (&o)[N]) const
    {
#pragma unroll
        for (int n = 0; n < N; n++) {
            Vec<4 * W> a;
#pragma unroll
            for (int k = 0; k < W; k++)
#pragma unroll
                for (int e = 0; e < 4; e++) a.w[4 * k + e] = v[n * W + k].w[e];
            o[n] = narrow<DT, 4>(a);
        }
    }
};

// Shape of a streaming launch.  G = operand tiles per ring stage: G = 1, a stage holds one tile of up to a whole
// stage; G = 2, tiles are half as long, a stage holds the tiles of two consecutive operations of the program,
// each brought by its own bulk copy, and is handed over once for both, so that the partial results that wait
// in the stack are half as large per tile while the bytes per stage hand-over stay the same.  CW = consumer
// warps: the 512 / G vectors of a tile are spread over CW * 32 threads, N = 16 / (G * CW) vectors each.  The
// path is bound by instruction issue as much as by HBM (the waits, releases and the decoding of an operation
// cost a warp about as many issue slots as the combines of two vectors), so fewer warps with more vectors
// each spend fewer slots per byte.
template <int G, int CW> struct StreamShape {
    static constexpr int CT = CW * 32;                       // consumer threads
    static constexpr int N = kStageVecs / (G * CT);          // vectors per thread and operand
    static constexpr int THREADS = CT + 32 * kProducers;
    static_assert(N >= 1 && N * G * CT == kStageVecs, "a tile is a whole number of vectors per consumer thread");
};
constexpr int kStreamBlocks = 3;    // thread blocks per SM the registers must leave room for (shared memory decides how many run)
// Whether the kernel evaluates the sub-expressions marked in the programs (bit 30) in a second accumulator, which
// saves their pushes and pops and one level of the shared-memory stack.  Not where a thread's accumulator is
// 32 registers already (16-bit elements on whole-stage tiles: these serve shallow programs only).
template <int DT, int G> struct SecondAccumulator { static constexpr bool value = !(Wide<DT>::half && G == 1); };

template <int DT, int OPR, typename PRM, int G, int CW>
__global__ void __launch_bounds__(StreamShape<G, CW>::THREADS, kStreamBlocks)
rd_tree_stream_kernel(const __grid_constant__ PRM a)
{
    using Jobs = typename PRM::Jobs;
    using Shape = StreamShape<G, CW>;
    constexpr int N = Shape::N;
    constexpr uint32_t CT = Shape::CT;
    constexpr uint32_t kStageBytes = kStageWords * 4u, kSubBytes = kStageBytes / uint32_t(G);
    constexpr uint32_t kLevelBytes = uint32_t(N) * uint32_t(Wide<DT>::W) * CT * 16u;          // one stack level
    constexpr uint32_t kSecondBit = 1u << (30 - kIdxBits), kMergeBit = 1u << (31 - kIdxBits); // in an operation word >> kIdxBits
    constexpr bool AUX = SecondAccumulator<DT, G>::value;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int S = a.stages;
    // dynamic shared memory: ring [S][G][kSubBytes] | stack [depth][N * W][CT] vectors | full[S] | empty[S] | steps [S][G]
    const uint32_t ring = smem_addr(smem_raw);
    const uint32_t stack = ring + uint32_t(S) * kStageBytes;
    const uint32_t full = stack + uint32_t(a.depth) * kLevelBytes;
    const uint32_t empty = full + uint32_t(S) * 8u;
    const uint32_t stepWords = empty + uint32_t(S) * 8u;             // per stage: the operation words of its G operands
    __shared__ int abort_flag;
    __shared__ TileQueue tileq;
    const uint32_t tid = threadIdx.x;

    if (tid == 0) {
        abort_flag = 0;
        tileq.published = 0;
        for (int s = 0; s < S; s++) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full + uint32_t(s) * 8u), "r"(1u) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty + uint32_t(s) * 8u), "r"(uint32_t(CW)) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Programmatic dependent launch: the next launch on the stream may begin while this grid is still running,
    // as soon as an SM has room for one of its thread blocks.  What does not depend on the grid before (barriers,
    // the tile counter, tile descriptors, operation words, source addresses: tables the host wrote) is done
    // right away; each thread waits for the grid before it to have finished completely just before its first
    // access to message data: the producers before their first copy, the consumers before their first store.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited = false;

    if (tid >= CT) {
        // ------------------------------------------------------------------ producers
        // One lane in each of the kProducers producer warps.  A step is one ring stage: the operand tiles of
        // G consecutive operations of a tile's program.  Producer j owns the steps j, j + P, j + 2P, ... of
        // this CTA's sequence of steps and issues them in order: stages are released by the consumers in that
        // same order, so a producer never waits for a stage while a later one of its own is already free.
        // Being alone in its warp, a producer polls without divergence; the table look-ups of a step are
        // issued before its wait.  The step's operation words travel to the consumers beside the stage.
        if ((tid & 31u) != 0) return;
        const int P = kProducers < S ? kProducers : S;
        const int j = int(tid - CT) / 32;
        if (j >= P) return;
        TileSource source;                      // used by producer 0 only
        if (j == 0) {
            uint32_t tile0 = 0, tile1 = 0;
            if (!a.tile_counter) a.tile_range(blockIdx.x, tile0, tile1);
            source.start(&tileq, a.tile_counter, tile0, tile1, a.total_tiles());
        }
        uint32_t k = 0;                         // position in this CTA's sequence of tiles
        uint32_t tile = j == 0 ? source.get(0) : tile_at(&tileq, 0, &abort_flag, a.status);
        Jobs jobs(a, tile, tile != kNoTile);
        int i = j;                              // step within the tile
        int p = jobs.p();                       // of the job `tile` belongs to
        int steps = (p + G - 1) / G;
        while (tile != kNoTile && i >= steps) {
            i -= steps; k++;
            tile = j == 0 ? source.get(k) : tile_at(&tileq, k, &abort_flag, a.status);
            if (tile != kNoTile) { jobs.seek(tile); p = jobs.p(); steps = (p + G - 1) / G; }
        }
        int stage = j % S;
        uint32_t laps = 0;                      // times this producer has gone round the ring
        uint32_t cur = 0xFFFFFFFFu;
        TileDesc td = TileDesc{0, 0, 0};
        bool ok = true, any = false;
        int lastStage = 0;
        uint32_t lastLap = 0;
        while (tile != kNoTile) {
            if (tile != cur) { td = jobs.tile(tile); cur = tile; }
            const int first = i * G;
            const int cnt = p - first < G ? p - first : G;
            uint32_t wv[G];
            const uint32_t *src[G];
#pragma unroll
            for (int g = 0; g < G; g++) {
                wv[g] = g < cnt ? __ldg(jobs.ops() + td.prog + first + g) : 0u;
                src[g] = g < cnt ? jobs.input(wv[g] & kIdxMask) + td.elem_off : nullptr;
            }
            if (laps >= 1u && !mbar_wait_at(empty + uint32_t(stage) * 8u, (laps - 1u) & 1u, &abort_flag)) { ok = false; break; }
            const uint32_t bytes = (td.len & kLenMask) * 4u;
            const uint32_t bar = full + uint32_t(stage) * 8u;
            if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
#pragma unroll
            for (int g = 0; g < G; g++)
                asm volatile("st.shared.u32 [%0], %1;" ::"r"(stepWords + uint32_t(stage * G + g) * 4u), "r"(wv[g]) : "memory");
            mbar_expect_tx_at(bar, bytes * uint32_t(cnt));             // (release: the words above are visible with the data)
#pragma unroll
            for (int g = 0; g < G; g++)
                if (g < cnt) bulk_load_at(ring + uint32_t(stage) * kStageBytes + uint32_t(g) * kSubBytes, src[g], bytes, bar);
            any = true; lastStage = stage; lastLap = laps;
            if (j == 0) source.poke(k);
            i += P;
            while (tile != kNoTile && i >= steps) {
                i -= steps; k++;
                tile = j == 0 ? source.get(k) : tile_at(&tileq, k, &abort_flag, a.status);
                if (tile != kNoTile) { jobs.seek(tile); p = jobs.p(); steps = (p + G - 1) / G; }
            }
            stage += P;
            if (stage >= S) { stage -= S; laps++; }
        }
        if (j == 0) source.finish(gridDim.x);
        if (!ok) {
            if (!abort_flag) { atomicCAS(a.status, 0, -5); abort_flag = 1; }
            // leave only after this producer's last copies have landed (bounded); its earlier ones were consumed
            if (any) {
                const long long start = clock64();
                while (!mbar_try_wait_at(full + uint32_t(lastStage) * 8u, lastLap & 1u) && clock64() - start < kWaitCycles) {}
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumers
    const uint32_t lane = tid & 31u;
    int stage = 0;
    uint32_t phase = 0;
    uint32_t k = 0;
    uint32_t tile = tile_at(&tileq, 0, &abort_flag, a.status);
    Jobs jobs(a, tile, tile != kNoTile);
    StageAcc<DT, N> top, side;      // the running value; the value of a sub-expression that needs no stack.  Every tile's
    top.clear();                    // program begins with a load, so nothing of a tile's values outlives the tile
    side.clear();
    for (; tile != kNoTile; tile = tile_at(&tileq, ++k, &abort_flag, a.status)) {
        jobs.seek(tile);
        const int p = jobs.p();
        const TileDesc td = jobs.tile(tile);
        const uint32_t len = td.len & kLenMask;                       // padded to whole 128-bit vectors
        uint32_t sp = stack;                                          // address of the next free stack level
        // The operations of a tile, G to a ring stage.  Most of them only combine their operand into the running value
        // (in the steady state of a pipelined schedule all but a few per tile do): those are taken by the inner loop,
        // which changes nothing but one of the two accumulators and the ring position; an operation that loads, pushes
        // or pops leaves the inner loop with its stage already in registers and is done by the general code below it.
        int i = 0;
        while (i < p) {
            uint32_t w[G];
            uint4 r[G][N];
            bool general = false;
            do {
                if (!mbar_wait_at(full + uint32_t(stage) * 8u, phase, &abort_flag)) {
                    if (!abort_flag) { atomicCAS(a.status, 0, -5); abort_flag = 1; }
                    return;
                }
                // the step's operation words, then its data: every thread reads its N vectors of each operand (threads
                // beyond a short tile's end read stale bytes of the stage and never store their results)
#pragma unroll
                for (int g = 0; g < G; g++)
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[g]) : "r"(stepWords + uint32_t(stage * G + g) * 4u) : "memory");
                const uint32_t stageAddr = ring + uint32_t(stage) * kStageBytes + tid * 16u;
#pragma unroll
                for (int g = 0; g < G; g++)
#pragma unroll
                    for (int n = 0; n < N; n++) r[g][n] = lds128(stageAddr + uint32_t(g) * kSubBytes + uint32_t(n) * CT * 16u);
                // the stage's data is in registers: hand the stage back to the producer
                __syncwarp();
                if (lane == 0) mbar_arrive_at(empty + uint32_t(stage) * 8u);
                if (++stage == S) { stage = 0; phase ^= 1u; }
                bool simple = G == 1;           // (two operations to a stage: the general code takes them, one after the other)
#pragma unroll
                for (int g = 0; g < G; g++) {
                    if (g > 0 && i + g >= p) break;
                    // combine the operand (incoming or held) into the running value, or into the sub-expression's, nothing popped
                    simple = simple && (((w[g] >> kIdxBits) & ~(AUX ? kSecondBit : 0u)) | 1u) == 3u;
                }
                if (!simple) { general = true; break; }
#pragma unroll
                for (int g = 0; g < G; g++) {
                    if (g > 0 && i + g >= p) break;
                    const bool held = Commutes<DT, OPR>::value || ((w[g] >> kIdxBits) & 1u) == 0u;   // max, min: else the operand is the held value
                    if (AUX && ((w[g] >> kIdxBits) & kSecondBit)) {
                        if (held) side.template accumulate<OPR, true>(r[g]);
                        else side.template accumulate<OPR, false>(r[g]);
                    } else {
                        if (held) top.template accumulate<OPR, true>(r[g]);
                        else top.template accumulate<OPR, false>(r[g]);
                    }
                }
                i += G;
            } while (i < p);
            if (!general) break;
#pragma unroll
            for (int g = 0; g < G; g++) {
                if (g > 0 && i + g >= p) break;
                const uint32_t ctl = w[g] >> kIdxBits;                // kind | pops << 2 | roles of the pops << 6 | hints << 18
                if (G > 1 && ((ctl & ~(AUX ? kSecondBit : 0u)) | 1u) == 3u) {
                    // the common step: combine into the running value, or into the sub-expression's, no pops
                    const bool held = Commutes<DT, OPR>::value || (ctl & 1u) == 0u;
                    if (AUX && (ctl & kSecondBit)) {
                        if (held) side.template accumulate<OPR, true>(r[g]);
                        else side.template accumulate<OPR, false>(r[g]);
                    } else {
                        if (held) top.template accumulate<OPR, true>(r[g]);
                        else top.template accumulate<OPR, false>(r[g]);
                    }
                    continue;
                }
                const uint32_t kind = ctl & 3u;
                uint32_t npop = (ctl >> 2) & 0xFu;
                uint32_t roles = ctl >> 6;
                if (AUX && (ctl & kSecondBit)) {
                    // a sub-expression that needs no stack: it is evaluated in `side`, the running value stays put
                    if (kind == 1u) side.load(r[g]);
                    else if (kind == 2u || Commutes<DT, OPR>::value) side.template accumulate<OPR, true>(r[g]);
                    else side.template accumulate<OPR, false>(r[g]);
                    if (!(ctl & kMergeBit)) continue;
                    // its end: what a stack machine would pop first is the running value, its current value is `side`
                    npop--;
                    const bool poppedHeld = (roles & 1u) != 0;
                    roles >>= 1;
                    if (poppedHeld || Commutes<DT, OPR>::value) top.template accumulate<OPR, true>(side);
                    else top.template accumulate<OPR, false>(side);
                } else {
                    if (kind == 1u) {
                        top.push(sp, tid, CT);
                        sp += kLevelBytes;
                    }
                    if (kind <= 1u) top.load(r[g]);
                    else if (kind == 2u || Commutes<DT, OPR>::value) top.template accumulate<OPR, true>(r[g]);
                    else top.template accumulate<OPR, false>(r[g]);
                }
                while (npop--) {
                    sp -= kLevelBytes;
                    const bool poppedHeld = (roles & 1u) != 0;
                    roles >>= 1;
                    if (poppedHeld || Commutes<DT, OPR>::value) top.template pop_accumulate<OPR, true>(sp, tid, CT);
                    else top.template pop_accumulate<OPR, false>(sp, tid, CT);
                }
            }
            i += G;
        }
        bool live[N];
#pragma unroll
        for (int n = 0; n < N; n++) live[n] = (uint32_t(n) * CT + tid) * 4u < len;
        Vec<4> res[N];
        top.result(res);
        // A segment may begin or end inside a vector: the tile then starts / ends with a vector whose other
        // elements belong to the neighbouring segment (another tile writes those); only this tile's are stored.
        uint32_t *dst = jobs.out() + td.elem_off;
        const uint32_t head = (td.len >> 16) & 3u, tail = (td.len >> 18) & 3u, lastVec = len / 4u - 1u;
        if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
#pragma unroll
        for (int n = 0; n < N; n++) {
            const uint32_t vec = uint32_t(n) * CT + tid;
            if (live[n]) store_part(dst + vec * 4u, res[n], vec == 0u ? head : 0u, vec == lastVec ? tail : 0u);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Direct variant (128-bit path, few processes).  With a handful of operands a tile is finished after a
// handful of ring hand-offs and the ring's per-stage cost, not HBM, sets the pace.  Here a thread
// fetches the vectors of all p operands of its elements at once, in program order, into registers
// (P * U independent 128-bit loads in flight per thread) and then runs the program on them; the
// partial results that have to wait (at most log2 P) sit in a register stack that is shifted on
// push and pop, so that every register index is static.  Works on the streaming variant's tiles.
// ---------------------------------------------------------------------------------------------
constexpr int kDirectThreads = 256;

template <int P> struct DirectShape;    // D = stack entries (log2 P), U = vectors per thread and pass, B = blocks per SM
template <> struct DirectShape<2> { static constexpr int D = 1, U = 2, B = 4; };
template <> struct DirectShape<4> { static constexpr int D = 2, U = 2, B = 3; };
template <> struct DirectShape<8> { static constexpr int D = 3, U = 1, B = 4; };

template <int DT, int OPR, int P>
__global__ void __launch_bounds__(kDirectThreads, DirectShape<P>::B)
rd_tree_direct_kernel(const __grid_constant__ TreeParams<true> a)
{
    constexpr int D = DirectShape<P>::D, U = DirectShape<P>::U;
    const uint32_t tid = threadIdx.x;
    const int p = a.p;
    // Programmatic dependent launch, as in the streaming variant: the next launch on the stream may start
    // its blocks and read its tables while this grid runs; message data is touched only after the grid
    // before this one has finished.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool waited = false;
    for (uint32_t tile = blockIdx.x; tile < a.n_tiles; tile += gridDim.x) {
        const TileDesc td = a.tiles[tile];
        const uint32_t *prog = a.ops + td.prog;
        const uint32_t len = td.len & kLenMask;                       // padded to whole 128-bit vectors
        const uint32_t head = (td.len >> 16) & 3u, tail = (td.len >> 18) & 3u, lastVec = len / 4u - 1u;
        uint32_t w[P];
#pragma unroll
        for (int k = 0; k < P; k++) w[k] = k < p ? __ldg(prog + k) : 0u;
        if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
        for (uint32_t v0 = 0; v0 * 4u < len; v0 += uint32_t(U) * kDirectThreads) {
            uint32_t vec[U];
            bool live[U];
#pragma unroll
            for (int u = 0; u < U; u++) { vec[u] = v0 + uint32_t(u) * kDirectThreads + tid; live[u] = vec[u] * 4u < len; }
            Vec<4> x[P][U];
#pragma unroll
            for (int k = 0; k < P; k++) {
                if (k < p) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(a.input(w[k] & kIdxMask) + td.elem_off);
#pragma unroll
                    for (int u = 0; u < U; u++) {
                        uint4 r = make_uint4(0, 0, 0, 0);
                        if (live[u]) r = __ldcs(src + vec[u]);
                        x[k][u].w[0] = r.x; x[k][u].w[1] = r.y; x[k][u].w[2] = r.z; x[k][u].w[3] = r.w;
                    }
                }
            }
            Vec<4> top[U], st[D][U];
#pragma unroll
            for (int u = 0; u < U; u++) {
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    top[u].w[e] = 0;
#pragma unroll
                    for (int d = 0; d < D; d++) st[d][u].w[e] = 0;
                }
            }
#pragma unroll
            for (int k = 0; k < P; k++) {
                if (k < p) {
                    const uint32_t kind = (w[k] >> kIdxBits) & 3u;
                    if (kind == 1u) {                      // PUSH_LOAD: the stack moves down one entry
#pragma unroll
                        for (int u = 0; u < U; u++) {
#pragma unroll
                            for (int d = D - 1; d > 0; d--) st[d][u] = st[d - 1][u];
                            st[0][u] = top[u];
                        }
                    }
                    if (kind <= 1u) {
#pragma unroll
                        for (int u = 0; u < U; u++) top[u] = x[k][u];
                    } else if (kind == 2u || Commutes<DT, OPR>::value) {
#pragma unroll
                        for (int u = 0; u < U; u++) combine_vec<DT, OPR, 4>(top[u], top[u], x[k][u]);
                    } else {
#pragma unroll
                        for (int u = 0; u < U; u++) combine_vec<DT, OPR, 4>(top[u], x[k][u], top[u]);
                    }
                    uint32_t npop = (w[k] >> (kIdxBits + 2)) & 0xFu;
                    uint32_t roles = w[k] >> (kIdxBits + 6);
                    while (npop--) {
                        const bool poppedHeld = (roles & 1u) != 0;
                        roles >>= 1;
#pragma unroll
                        for (int u = 0; u < U; u++) {
                            const Vec<4> y = st[0][u];
#pragma unroll
                            for (int d = 0; d + 1 < D; d++) st[d][u] = st[d + 1][u];
                            if (poppedHeld || Commutes<DT, OPR>::value) combine_vec<DT, OPR, 4>(top[u], y, top[u]);
                            else combine_vec<DT, OPR, 4>(top[u], top[u], y);
                        }
                    }
                }
            }
            uint32_t *dst = a.out + td.elem_off;
#pragma unroll
            for (int u = 0; u < U; u++)
                if (live[u]) store_part(dst + vec[u] * 4u, top[u], vec[u] == 0u ? head : 0u, vec[u] == lastVec ? tail : 0u);
        }
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
    const size_t smem = size_t(depth) * kU * kTreeThreads * sizeof(Vec<V * Wide<DT>::W>);
    cudaError_t e = opt_in_shared_memory(reinterpret_cast<const void *>(kernel), l.device);
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
    constexpr int V = ElemWords<DT>::value;              // one element per thread and load
    return l.p <= kPackedPtrs ? launch_one<DT, OPR, V, true>(l) : launch_one<DT, OPR, V, false>(l);
}

// Launches the streaming kernel for one parameter type (one job with packed pointers, one job with a
// pointer table, or a batch) and one shape (operand tiles per ring stage, consumer warps).
template <int DT, int OPR, int G, int CW, typename PRM>
cudaError_t launch_stream_kernel(const PRM &prm, uint32_t n_ctas, int device, void *stream)
{
    auto kernel = rd_tree_stream_kernel<DT, OPR, PRM, G, CW>;
    const size_t smem = stream_smem_bytes(prm.stages, prm.depth, kStageWords, Wide<DT>::W, G);
    if (cudaError_t e = opt_in_shared_memory(reinterpret_cast<const void *>(kernel), device)) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ctas); cfg.blockDim = dim3(StreamShape<G, CW>::THREADS); cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, prm);
}
template <int DT, int OPR, typename PRM>
cudaError_t launch_stream_kernel(const PRM &prm, int ops_per_stage, int consumer_warps, uint32_t n_ctas, int device, void *stream)
{
    if (ops_per_stage == 2 && consumer_warps == 4) return launch_stream_kernel<DT, OPR, 2, 4>(prm, n_ctas, device, stream);
    if (ops_per_stage == 1 && consumer_warps == 4) return launch_stream_kernel<DT, OPR, 1, 4>(prm, n_ctas, device, stream);
    if constexpr (!Wide<DT>::half)       // (elements widened to fp32 always run with four consumer warps)
        if (ops_per_stage == 1 && consumer_warps == 8) return launch_stream_kernel<DT, OPR, 1, 8>(prm, n_ctas, device, stream);
    return cudaErrorInvalidValue;
}

template <int DT, int OPR, bool PACKED>
cudaError_t launch_stream(const TreeLaunch &l)
{
    StreamParams<PACKED> prm;
    if constexpr (PACKED) {
        for (int i = 0; i < kPackedPtrs; i++) prm.t.in.ptr[i] = i < l.p ? static_cast<const uint32_t *>(l.host_ptrs[i]) : nullptr;
    } else {
        prm.t.in.table = reinterpret_cast<const uint32_t *const *>(l.dev_ptr_table);
    }
    prm.t.out = static_cast<uint32_t *>(l.out);
    prm.t.tiles = l.tiles; prm.t.ops = l.ops; prm.t.n_tiles = l.n_tiles; prm.t.p = l.p;
    prm.cta_first = l.cta_first; prm.status = l.status; prm.tile_counter = l.tile_counter;
    prm.stages = l.stages; prm.depth = l.shared_depth > 0 ? l.shared_depth : 1;
    return launch_stream_kernel<DT, OPR>(prm, l.ops_per_stage, l.consumer_warps, l.n_ctas, l.device, l.stream);
}

template <int DT, int OPR>
cudaError_t launch_stream_batch(const BatchLaunch &b)
{
    const int depth = b.stack_depth > 0 ? b.stack_depth : 1;
    if (b.host_jobs) {
        BatchStreamParams<true> prm;
        for (uint32_t j = 0; j < uint32_t(kBatchPackJobs); j++)
            prm.jobs[j] = j < b.n_jobs ? b.host_jobs[j] : BatchJob{nullptr, nullptr, nullptr, nullptr, b.n_tiles, b.n_tiles, 1, 0};
        for (uint32_t i = 0; i < uint32_t(kBatchPackPtrs); i++)
            prm.ptrs[i] = i < b.n_ptrs ? static_cast<const uint32_t *>(b.host_ptrs[i]) : nullptr;
        prm.n_jobs = b.n_jobs; prm.n_tiles = b.n_tiles; prm.status = b.status; prm.tile_counter = b.tile_counter;
        prm.stages = b.stages; prm.depth = depth;
        return launch_stream_kernel<DT, OPR>(prm, b.ops_per_stage, b.consumer_warps, b.n_ctas, b.device, b.stream);
    }
    BatchStreamParams<false> prm;
    prm.jobs = b.jobs; prm.n_jobs = b.n_jobs; prm.n_tiles = b.n_tiles; prm.status = b.status; prm.tile_counter = b.tile_counter;
    prm.stages = b.stages; prm.depth = depth;
    return launch_stream_kernel<DT, OPR>(prm, b.ops_per_stage, b.consumer_warps, b.n_ctas, b.device, b.stream);
}

template <int DT, int OPR>
cudaError_t launch_stream_dtop(const TreeLaunch &l)
{
    return l.p <= kPackedPtrs ? launch_stream<DT, OPR, true>(l) : launch_stream<DT, OPR, false>(l);
}

template <int DT, int OPR, int P>
cudaError_t launch_direct(const TreeLaunch &l)
{
    TreeParams<true> prm;
    for (int i = 0; i < kPackedPtrs; i++) prm.in.ptr[i] = i < l.p ? static_cast<const uint32_t *>(l.host_ptrs[i]) : nullptr;
    prm.out = static_cast<uint32_t *>(l.out);
    prm.tiles = l.tiles; prm.ops = l.ops; prm.n_tiles = l.n_tiles; prm.p = l.p;
    uint32_t grid = uint32_t(l.sm_count) * uint32_t(DirectShape<P>::B);
    if (grid > l.n_tiles) grid = l.n_tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kDirectThreads); cfg.dynamicSmemBytes = 0;
    cfg.stream = static_cast<cudaStream_t>(l.stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rd_tree_direct_kernel<DT, OPR, P>, prm);
}

template <int DT, int OPR>
cudaError_t launch_direct_dtop(const TreeLaunch &l)
{
    if (l.p <= 2) return launch_direct<DT, OPR, 2>(l);
    if (l.p <= 4) return launch_direct<DT, OPR, 4>(l);
    return launch_direct<DT, OPR, 8>(l);
}

// Calls f.template operator()<DT, OPR>() for the run-time operation.
template <int DT, typename F> cudaError_t with_op(int op, F &&f)
{
    if constexpr (DT == DT_BF16_PICK || DT == DT_FP16_PICK) {        // these serve max and min only
        return op == OPR_MAX ? f.template operator()<DT, OPR_MAX>() : op == OPR_MIN ? f.template operator()<DT, OPR_MIN>() : cudaErrorInvalidValue;
    }
    switch (op) {
    case OPR_SUM: return f.template operator()<DT, OPR_SUM>();
    case OPR_MAX: return f.template operator()<DT, OPR_MAX>();
    case OPR_MIN: return f.template operator()<DT, OPR_MIN>();
    default: return f.template operator()<DT, OPR_PROD>();
    }
}
struct StreamLauncher {
    const TreeLaunch &l;
    template <int DT, int OPR> cudaError_t operator()() const { return launch_stream_dtop<DT, OPR>(l); }
};
struct BatchLauncher {
    const BatchLaunch &b;
    template <int DT, int OPR> cudaError_t operator()() const { return launch_stream_batch<DT, OPR>(b); }
};
struct DirectLauncher {
    const TreeLaunch &l;
    template <int DT, int OPR> cudaError_t operator()() const
    {
        if constexpr (DT >= DT_BF16) return cudaErrorInvalidValue;       // 16-bit types go through the streaming kernel
        else return launch_direct_dtop<DT, OPR>(l);
    }
};
struct ElementLauncher {
    const TreeLaunch &l;
    template <int DT, int OPR> cudaError_t operator()() const { return launch_dtop<DT, OPR>(l); }
};

}  // namespace

// This file is compiled once per element type (RD_DT = 0..5: that type's kernels behind one entry point)
// and once without RD_DT (launch shapes and the dispatch over the element types), so that the element
// types build side by side.
#ifdef RD_DT

#define RD_CAT2(a, b) a##b
#define RD_CAT(a, b) RD_CAT2(a, b)
int RD_CAT(launch_for_dtype_, RD_DT)(int which, const void *launch, int op)
{
    switch (which) {
    case LAUNCH_STREAM: return int(with_op<RD_DT>(op, StreamLauncher{*static_cast<const TreeLaunch *>(launch)}));
    case LAUNCH_BATCH: return int(with_op<RD_DT>(op, BatchLauncher{*static_cast<const BatchLaunch *>(launch)}));
    case LAUNCH_DIRECT: return int(with_op<RD_DT>(op, DirectLauncher{*static_cast<const TreeLaunch *>(launch)}));
    default: return int(with_op<RD_DT>(op, ElementLauncher{*static_cast<const TreeLaunch *>(launch)}));
    }
}

#else

uint32_t tree_tile_elems(int vec) { return uint32_t(kTreeThreads) * kU * uint32_t(vec); }

// One stack level holds the partial results of one tile.  (acc_words: words of partial result per message word,
// 2 for the 16-bit types, whose elements are combined in fp32, else 1; ops_per_stage: operand tiles that share a
// ring stage, each stage_elems / ops_per_stage words long.)
static int stack_level_bytes(int stage_elems, int acc_words, int ops_per_stage)
{
    return stage_elems / ops_per_stage * acc_words * 4;
}

size_t stream_smem_bytes(int stages, int depth, int stage_elems, int acc_words, int ops_per_stage)
{
    // ring | stack | two barriers per stage | the operation words of a stage's operands
    return size_t(stages) * size_t(stage_elems) * 4 + size_t(depth) * stack_level_bytes(stage_elems, acc_words, ops_per_stage) +
           size_t(2 * stages) * sizeof(uint64_t) + size_t(stages) * size_t(ops_per_stage) * sizeof(uint32_t);
}

int stream_stage_elems(uint64_t elems_per_cta)
{
    // Measured on B200: the time per stage hand-over hardly depends on the stage's size up to 8 KB, so smaller
    // stages only lower the throughput, also for small messages.
    (void)elems_per_cta;
    return kStageWords;
}

bool stream_second_accumulator(int acc_words, int ops_per_stage) { return !(acc_words > 1 && ops_per_stage == 1); }

void stream_shape(int stack_depth, int acc_words, int ops_per_stage, bool many_pushes, int smem_per_sm, int stage_elems, uint64_t n_tiles,
                  int sm_count, int *ctas_per_sm, int *stages)
{
    const int depth = stack_depth > 0 ? stack_depth : 1;
    const int stageBytes = stage_elems * 4;
    // Stages that fit when `ctas` CTAs share an SM (room left for the per-CTA reserve and statics).
    auto fit = [&](int ctas) {
        return (smem_per_sm / ctas - 2048 - depth * stack_level_bytes(stage_elems, acc_words, ops_per_stage) - 512) / stageBytes;
    };
    // Measured on B200: with many tiles per CTA, three CTAs with 4 stages each stream 3-7 % more than two
    // with 6 to 13 (6.8-7.0 TB/s for 3 to 256 processes); the bytes in flight are no more, the third set
    // of consumers is what helps (three CTAs with 5 stages are behind 4, and 3 stages are too few to hide
    // the hand-off).  With few tiles the count of tiles per CTA decides instead: every CTA of an SM gets
    // 1 / ctas of its bandwidth, so a launch lasts about ceil(tiles / CTAs) * ctas tile times.  Three CTAs
    // are chosen when their product is at most 8 % above that of two (512 tiles on 148 SMs: 2 * 3 against
    // 2 * 2, two CTAs are 20 % faster; 768 tiles: 2 * 3 against 3 * 2, three are 4 % faster; 1024 tiles:
    // 3 * 3 against 4 * 2, two are 3 % faster).  Two CTAs take all the stages that fit: a launch of one or
    // two tiles per CTA is over sooner the more of it is in flight from the start.
    const int s3 = fit(3), s2 = fit(2);
    // The 16-bit types under sum and product (fp32 partial results, two tiles per stage) spend the most issue slots
    // per byte and gain from a third thread block even when it leaves only three stages each, or two where the
    // programs push often (binomial-like trees).  Measured, bf16 sum, 64 MiB messages, GB/s: three blocks x 3
    // stages against two x 6, p = 256 (six levels of stack): uni-greedy 7035 / 6828, binomial 6294 / 5473; three
    // blocks x 2 stages against two x 6, p = 512 (seven levels): uni-greedy 6318 / 6599, binomial 6005 / 5418.
    if (acc_words > 1 && sm_count > 0 && (s3 == 3 || (s3 == 2 && many_pushes))) { *ctas_per_sm = 3; *stages = s3; return; }
    if (s3 >= 4 && s2 >= 3 && sm_count > 0) {
        const uint64_t t = n_tiles > 0 ? n_tiles : 1;
        const uint64_t cost3 = (t + 3u * uint64_t(sm_count) - 1) / (3u * uint64_t(sm_count)) * 3u;
        const uint64_t cost2 = (t + 2u * uint64_t(sm_count) - 1) / (2u * uint64_t(sm_count)) * 2u;
        if (cost3 * 100u <= cost2 * 108u) { *ctas_per_sm = 3; *stages = 4; return; }
    }
    // Two CTAs per SM whenever each still gets three stages (deep stacks, p = 512..1024: two CTAs with
    // 4-5 stages stream 6.6 TB/s where one CTA with 19 stages reaches 5.3).
    if (s2 >= 3) { *ctas_per_sm = 2; *stages = s2 > kMaxStages ? kMaxStages : s2; return; }
    const int s1 = fit(1);
    *ctas_per_sm = 1;
    *stages = s1 > kMaxStages ? kMaxStages : s1 < 2 ? 2 : s1;
}

int launch_for_dtype_0(int which, const void *launch, int op);
int launch_for_dtype_1(int which, const void *launch, int op);
int launch_for_dtype_2(int which, const void *launch, int op);
int launch_for_dtype_3(int which, const void *launch, int op);
int launch_for_dtype_4(int which, const void *launch, int op);
int launch_for_dtype_5(int which, const void *launch, int op);
int launch_for_dtype_6(int which, const void *launch, int op);
int launch_for_dtype_7(int which, const void *launch, int op);

static int launch_for(int dtype, int which, const void *launch, int op)
{
    if ((dtype == DT_BF16 || dtype == DT_FP16) && (op == OPR_MAX || op == OPR_MIN)) dtype += DT_BF16_PICK - DT_BF16;
    switch (dtype) {
    case DT_INT32: return launch_for_dtype_0(which, launch, op);
    case DT_FP32: return launch_for_dtype_1(which, launch, op);
    case DT_INT64: return launch_for_dtype_2(which, launch, op);
    case DT_FP64: return launch_for_dtype_3(which, launch, op);
    case DT_BF16: return launch_for_dtype_4(which, launch, op);
    case DT_FP16: return launch_for_dtype_5(which, launch, op);
    case DT_BF16_PICK: return launch_for_dtype_6(which, launch, op);
    default: return launch_for_dtype_7(which, launch, op);
    }
}

int launch_tree_stream(const TreeLaunch &l)
{
    if (l.n_tiles == 0 || l.n_ctas == 0) return 0;
    return launch_for(l.dtype, LAUNCH_STREAM, &l, l.op);
}

int launch_tree_stream_batch(const BatchLaunch &b)
{
    if (b.n_jobs == 0 || b.n_ctas == 0) return 0;
    return launch_for(b.dtype, LAUNCH_BATCH, &b, b.op);
}

bool direct_applies(int p, int stack_depth)
{
    if (p > kDirectMaxProcs) return false;
    return stack_depth <= (p <= 2 ? 1 : p <= 4 ? 2 : 3);   // DirectShape<P>::D of the instantiation that serves p
}

int direct_blocks_per_sm(int p) { return p <= 2 ? DirectShape<2>::B : p <= 4 ? DirectShape<4>::B : DirectShape<8>::B; }

int launch_tree_direct(const TreeLaunch &l)
{
    if (l.n_tiles == 0) return 0;
    return launch_for(l.dtype, LAUNCH_DIRECT, &l, l.op);
}

int launch_tree(const TreeLaunch &l)
{
    if (l.n_tiles == 0) return 0;
    return launch_for(l.dtype, LAUNCH_ELEMENT, &l, l.op);
}

#endif  // RD_DT

}  // namespace rd
