// Schedule-faithful execution on sm_100a: groups of thread blocks play the processes.
//
// Process i is played by G thread blocks ("lanes"); lane g owns the same range of words of every
// scratch slot (1/G of it), so the G lanes are G independent copies of the
// whole p-process system working on disjoint parts of the message and of the scratch slots, and
// never synchronise with each other.  Each block walks its process's
// action list in order:
//   send     post a flag for the pair (release), so that the receiver may read the value this
//            process holds for the segment (its input, or its partial result in a scratch slot);
//            with one port per process the sender then waits until the receiver has taken it.
//   receive  wait for the sender's flag (acquire), read the sender's value, combine it with the value
//            held here (held operand first) or just store it, write the result to this process's
//            slot (the root: to the output), then raise the pair's "taken" flag.
// Flags carry the launch's epoch number, so they never need clearing.  Every wait is bounded by a
// clock budget: when it runs out the block records RD_ERR_TIMEOUT, raises a global abort flag that
// all other waits watch, and leaves; nothing traps and nothing spins forever.
// All blocks must be resident at once (cooperative launch).
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "rd_kernels.h"

namespace rd {

namespace {

enum { DT_INT32 = 0, DT_FP32 = 1, DT_INT64 = 2, DT_FP64 = 3 };

// Buffers are indexed in 32-bit words; an element is one word or two.
template <int DT> struct ElemWords { static constexpr int value = DT >= DT_INT64 ? 2 : 1; };
enum { OPR_SUM = 0, OPR_MAX = 1, OPR_MIN = 2, OPR_PROD = 3 };

template <int DT, int OPR> __device__ __forceinline__ uint32_t combine(uint32_t held, uint32_t in)
{
    if (DT == DT_INT32) {
        if (OPR == OPR_SUM) return held + in;
        if (OPR == OPR_PROD) return held * in;
        if (OPR == OPR_MAX) return (int32_t(in) > int32_t(held)) ? in : held;
        return (int32_t(in) < int32_t(held)) ? in : held;
    } else {
        const float h = __uint_as_float(held), i = __uint_as_float(in);
        if (OPR == OPR_SUM) return __float_as_uint(__fadd_rn(h, i));
        if (OPR == OPR_PROD) return __float_as_uint(__fmul_rn(h, i));
        if (OPR == OPR_MAX) return (i > h) ? in : held;
        return (i < h) ? in : held;
    }
}

template <int DT, int OPR> __device__ __forceinline__ unsigned long long combine64(unsigned long long held, unsigned long long in)
{
    if (DT == DT_INT64) {
        if (OPR == OPR_SUM) return held + in;
        if (OPR == OPR_PROD) return held * in;
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

// V words as one access (V = 1, 2 or 4) through L2, where the other blocks' stores are visible.
template <int V> struct Words { uint32_t w[V]; };
template <int V> __device__ __forceinline__ Words<V> load_words(const uint32_t *p)
{
    Words<V> r;
    if constexpr (V == 4) { const uint4 t = __ldcg(reinterpret_cast<const uint4 *>(p)); r.w[0] = t.x; r.w[1] = t.y; r.w[2] = t.z; r.w[3] = t.w; }
    else if constexpr (V == 2) { const uint2 t = __ldcg(reinterpret_cast<const uint2 *>(p)); r.w[0] = t.x; r.w[1] = t.y; }
    else r.w[0] = __ldcg(p);
    return r;
}
template <int V> __device__ __forceinline__ void store_words(uint32_t *p, const Words<V> &v)
{
    if constexpr (V == 4) __stcg(reinterpret_cast<uint4 *>(p), make_uint4(v.w[0], v.w[1], v.w[2], v.w[3]));
    else if constexpr (V == 2) __stcg(reinterpret_cast<uint2 *>(p), make_uint2(v.w[0], v.w[1]));
    else __stcg(p, v.w[0]);
}
template <int DT, int OPR, int V> __device__ __forceinline__ Words<V> combine_words(const Words<V> &held, const Words<V> &in)
{
    Words<V> r;
    if constexpr (ElemWords<DT>::value == 1) {
#pragma unroll
        for (int v = 0; v < V; v++) r.w[v] = combine<DT, OPR>(held.w[v], in.w[v]);
    } else {
        static_assert(V % 2 == 0, "an 8-byte element is never split between two accesses");
#pragma unroll
        for (int v = 0; v < V; v += 2) {
            const unsigned long long h = (unsigned long long)held.w[v] | ((unsigned long long)held.w[v + 1] << 32);
            const unsigned long long i = (unsigned long long)in.w[v] | ((unsigned long long)in.w[v + 1] << 32);
            const unsigned long long c = combine64<DT, OPR>(h, i);
            r.w[v] = uint32_t(c); r.w[v + 1] = uint32_t(c >> 32);
        }
    }
    return r;
}

__device__ __forceinline__ unsigned long long now_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint32_t load_acquire(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void store_release(uint32_t *p, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Thread 0 waits until *flag == epoch; everybody learns the outcome.  False: gave up or aborted.
__device__ __forceinline__ bool wait_flag(const uint32_t *flag, uint32_t epoch, const FaithfulParams &a, int *sh_ok)
{
    if (threadIdx.x == 0) {
        int ok = 1;
        if (load_acquire(flag) != epoch) {
            const long long start = clock64();
            uint32_t turns = 0;
            while (load_acquire(flag) != epoch) {
                __nanosleep(40);
                if ((++turns & 15u) == 0u) {
                    if (*reinterpret_cast<volatile int *>(a.abort_flag) != 0) { ok = 0; break; }
                    if (clock64() - start > a.wait_cycles) {
                        atomicCAS(a.status, 0, -5);
                        atomicExch(a.abort_flag, 1);
                        ok = 0;
                        break;
                    }
                }
            }
        }
        *sh_ok = ok;
    }
    __syncthreads();
    const bool ok = *sh_ok != 0;
    __syncthreads();
    return ok;
}

template <int DT, int OPR, int V>
__global__ void __launch_bounds__(kFaithfulThreads, 8)
rd_faithful_kernel(const FaithfulParams a)
{
    __shared__ int sh_ok;
    const int proc = int(blockIdx.x) / a.lanes, lane = int(blockIdx.x) % a.lanes;
    const uint32_t k0 = a.first[proc], k1 = a.first[proc + 1];
    const uint32_t *mine = a.inputs[proc];
    unsigned long long t_begin = 0, t_end = 0;
    if (threadIdx.x == 0) t_begin = now_ns();
    bool alive = true;
    for (uint32_t k = k0; k < k1 && alive; k++) {
        const FaithfulAction act = a.actions[k];
        uint32_t *posted = a.posted + size_t(act.event) * a.lanes + lane;
        uint32_t *taken = a.taken + size_t(act.event) * a.lanes + lane;
        if (act.kind == 2) {
            // everything this block wrote for the segment is ordered before the flag
            __syncthreads();
            if (threadIdx.x == 0) { __threadfence(); store_release(posted, a.epoch); }
            if (a.blocking_send) alive = wait_flag(taken, a.epoch, a, &sh_ok);
            continue;
        }
        unsigned long long t_ready = 0, t_start = 0;
        if (threadIdx.x == 0 && lane == 0) t_ready = now_ns();
        if (act.wait_event >= 0)
            alive = wait_flag(a.taken + size_t(act.wait_event) * a.lanes + lane, a.epoch, a, &sh_ok);
        if (alive) alive = wait_flag(posted, a.epoch, a, &sh_ok);
        if (!alive) break;
        if (threadIdx.x == 0 && lane == 0) t_start = now_ns();
        // A segment that starts at word b of the message sits in its slot from word (b mod 4) on, so that
        // slot, messages and output agree on where the 128-bit boundaries fall and whole vectors can be
        // moved wherever a segment starts.  This lane's share is the same range of SLOT words for every
        // segment (a fixed 1/G of the slot): lanes run independently of each other and share the slots,
        // so a lane that is already re-using a slot for a later segment must never touch words that
        // belong to another lane's share of the segment still held there.
        const uint64_t seg_lo = a.seg_off[act.seg], seg_len = a.seg_off[act.seg + 1] - seg_lo;
        const uint64_t phase = seg_lo & 3u, first = phase, last = phase + seg_len;      // the segment's slot words
        const uint64_t units = a.slot_elems / V;
        uint64_t lo = units * uint64_t(lane) / uint64_t(a.lanes) * V;
        uint64_t hi = units * uint64_t(lane + 1) / uint64_t(a.lanes) * V;
        if (hi > (last + V - 1) / V * V) hi = (last + V - 1) / V * V;
        // all three pointers are indexed by slot word
        const uint32_t *src = act.peer_slot >= 0 ? a.scratch + (size_t(act.peer) * a.slots + size_t(act.peer_slot)) * a.slot_elems
                              : (act.peer_slot == -1 ? a.inputs[act.peer] : a.out) + (seg_lo - phase);
        uint32_t *dst = act.slot >= 0 ? a.scratch + (size_t(proc) * a.slots + size_t(act.slot)) * a.slot_elems : a.out + (seg_lo - phase);
        const uint32_t *held = act.first ? mine + (seg_lo - phase) : dst;
        const bool store_only = act.kind == 1;
        constexpr int E = ElemWords<DT>::value;
        for (uint64_t w = lo + uint64_t(threadIdx.x) * V; w < hi; w += uint64_t(kFaithfulThreads) * V) {
            if (w >= first && w + V <= last) {
                const Words<V> in = load_words<V>(src + w);
                store_words<V>(dst + w, store_only ? in : combine_words<DT, OPR, V>(load_words<V>(held + w), in));
            } else {
                // the vector holding the segment's first or last words: element by element
#pragma unroll
                for (int k = 0; k < V; k += E) {
                    if (w + k >= first && w + k < last) {
                        const Words<E> in = load_words<E>(src + w + k);
                        store_words<E>(dst + w + k, store_only ? in : combine_words<DT, OPR, E>(load_words<E>(held + w + k), in));
                    }
                }
            }
        }
        // the sender's value has been read: tell it
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            store_release(taken, a.epoch);
            t_end = now_ns();
            if (lane == 0) {
                a.trace[size_t(act.event) * 3 + 0] = t_ready;
                a.trace[size_t(act.event) * 3 + 1] = t_start;
                a.trace[size_t(act.event) * 3 + 2] = t_end;
            }
        }
    }
    if (threadIdx.x == 0) {
        if (t_end == 0) t_end = now_ns();
        a.block_times[size_t(blockIdx.x) * 2 + 0] = t_begin;
        a.block_times[size_t(blockIdx.x) * 2 + 1] = t_end;
    }
}

template <int DT, int OPR>
cudaError_t launch_dtop(const FaithfulParams &prm, bool wide, cudaStream_t stream, bool occupancy_only, int *blocks_per_sm)
{
    constexpr int N = ElemWords<DT>::value;      // narrow variant: one element per access
    const void *fn = wide ? reinterpret_cast<const void *>(rd_faithful_kernel<DT, OPR, 4>)
                          : reinterpret_cast<const void *>(rd_faithful_kernel<DT, OPR, N>);
    if (occupancy_only) {
        return wide ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, rd_faithful_kernel<DT, OPR, 4>, kFaithfulThreads, 0)
                    : cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, rd_faithful_kernel<DT, OPR, N>, kFaithfulThreads, 0);
    }
    FaithfulParams copy = prm;
    void *args[] = {&copy};
    return cudaLaunchCooperativeKernel(fn, dim3(unsigned(prm.n_procs * prm.lanes)), dim3(kFaithfulThreads), args, 0, stream);
}

template <int DT>
cudaError_t dispatch_op(const FaithfulParams &prm, int op, bool wide, cudaStream_t stream, bool occ, int *bps)
{
    return op == OPR_SUM ? launch_dtop<DT, OPR_SUM>(prm, wide, stream, occ, bps)
           : op == OPR_MAX ? launch_dtop<DT, OPR_MAX>(prm, wide, stream, occ, bps)
           : op == OPR_MIN ? launch_dtop<DT, OPR_MIN>(prm, wide, stream, occ, bps)
                           : launch_dtop<DT, OPR_PROD>(prm, wide, stream, occ, bps);
}

cudaError_t dispatch(const FaithfulParams &prm, int dtype, int op, bool wide, cudaStream_t stream, bool occ, int *bps)
{
    return dtype == DT_INT32 ? dispatch_op<DT_INT32>(prm, op, wide, stream, occ, bps)
           : dtype == DT_FP32 ? dispatch_op<DT_FP32>(prm, op, wide, stream, occ, bps)
           : dtype == DT_INT64 ? dispatch_op<DT_INT64>(prm, op, wide, stream, occ, bps)
                               : dispatch_op<DT_FP64>(prm, op, wide, stream, occ, bps);
}

}  // namespace

int faithful_blocks_per_sm(int dtype, int op, bool wide, int *blocks_per_sm)
{
    FaithfulParams dummy{};
    return int(dispatch(dummy, dtype, op, wide, nullptr, true, blocks_per_sm));
}

int launch_faithful(const FaithfulParams &prm, int dtype, int op, bool wide, void *stream)
{
    return int(dispatch(prm, dtype, op, wide, static_cast<cudaStream_t>(stream), false, nullptr));
}

// ---------------------------------------------------------------------------------------------
// The same kernel for callers that cannot allocate device memory: every table, flag and partial
// result lives in one file-scope device array of fixed size instead of cudaMalloc'ed buffers.
// In host code the array's name only stands for the symbol; the device address is asked for once
// per device (cudaGetSymbolAddress, with that device current) and handed to the kernel as ordinary
// pointers.  All calls share the array and it keeps what the last call left in it, so the flags,
// the status words and the time stamps are cleared at the start of every call.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = size_t(32) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

unsigned char *g_static_base[64] = {};   // per device: address of g_static_scratch once looked up
std::mutex g_static_base_lock;

size_t carve(size_t &cursor, size_t bytes)
{
    const size_t at = cursor;
    cursor += (bytes + 255) / 256 * 256;
    return at;
}

}  // namespace

size_t faithful_static_capacity() { return kStaticScratchBytes; }

int faithful_static_run(StaticRun &r)
{
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return 1;
    unsigned char *base = nullptr;
    {
        std::lock_guard<std::mutex> hold(g_static_base_lock);
        if (!g_static_base[device]) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return 1;
            g_static_base[device] = static_cast<unsigned char *>(ptr);
        }
        base = g_static_base[device];
    }
    // blocks per process: everything must be resident at once
    int perSm = 0, sms = 0, khz = 0;
    if (dispatch(FaithfulParams{}, r.dtype, r.op, r.wide, nullptr, true, &perSm) != cudaSuccess) return 1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return 1;
    if (cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, device) != cudaSuccess) return 1;
    const long long capacity = (long long)perSm * sms;
    if (capacity < r.p) return 3;
    const int lanes = int(capacity / r.p < 16 ? capacity / r.p : 16);
    // carve the array
    size_t cursor = 0;
    const size_t oActions = carve(cursor, r.n_actions * sizeof(FaithfulAction));
    const size_t oFirst = carve(cursor, size_t(r.p + 1) * sizeof(uint32_t));
    const size_t oSegOff = carve(cursor, r.n_seg_off * sizeof(uint64_t));
    const size_t oInputs = carve(cursor, size_t(r.p) * sizeof(void *));
    const size_t flagBytes = 2 * r.n_events * size_t(lanes) * sizeof(uint32_t);
    const size_t oFlags = carve(cursor, flagBytes);
    const size_t traceBytes = 3 * r.n_events * sizeof(unsigned long long);
    const size_t oTrace = carve(cursor, traceBytes);
    const size_t timeBytes = 2 * size_t(r.p) * size_t(lanes) * sizeof(unsigned long long);
    const size_t oTimes = carve(cursor, timeBytes);
    const size_t oStatus = carve(cursor, 2 * sizeof(int));
    const size_t oSlots = carve(cursor, size_t(r.p) * size_t(r.slots) * size_t(r.slot_elems) * sizeof(uint32_t));
    r.needed_bytes = cursor;
    if (cursor > kStaticScratchBytes) return 2;
    cudaStream_t stream = static_cast<cudaStream_t>(r.stream);
    bool ok = true;
    ok = ok && cudaMemcpyAsync(base + oActions, r.h_actions, r.n_actions * sizeof(FaithfulAction), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(base + oFirst, r.h_first, size_t(r.p + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(base + oSegOff, r.h_seg_off, r.n_seg_off * sizeof(uint64_t), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(base + oInputs, r.h_inputs, size_t(r.p) * sizeof(void *), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    // what must start at zero: flags (the array still holds the previous call's), status, abort flag, time stamps
    ok = ok && cudaMemsetAsync(base + oFlags, 0, flagBytes > 0 ? flagBytes : 4, stream) == cudaSuccess;
    ok = ok && cudaMemsetAsync(base + oTrace, 0, traceBytes > 0 ? traceBytes : 8, stream) == cudaSuccess;
    ok = ok && cudaMemsetAsync(base + oStatus, 0, 2 * sizeof(int), stream) == cudaSuccess;
    if (!ok) return 1;
    FaithfulParams prm{};
    prm.inputs = reinterpret_cast<const uint32_t *const *>(base + oInputs);
    prm.out = static_cast<uint32_t *>(r.d_out);
    prm.scratch = reinterpret_cast<uint32_t *>(base + oSlots);
    prm.actions = reinterpret_cast<const FaithfulAction *>(base + oActions);
    prm.first = reinterpret_cast<const uint32_t *>(base + oFirst);
    prm.seg_off = reinterpret_cast<const uint64_t *>(base + oSegOff);
    prm.posted = reinterpret_cast<uint32_t *>(base + oFlags);
    prm.taken = prm.posted + r.n_events * size_t(lanes);
    prm.trace = reinterpret_cast<unsigned long long *>(base + oTrace);
    prm.block_times = reinterpret_cast<unsigned long long *>(base + oTimes);
    prm.status = reinterpret_cast<int *>(base + oStatus);
    prm.abort_flag = prm.status + 1;
    prm.wait_cycles = (long long)(r.wait_seconds * double(khz > 0 ? khz : 1000000) * 1e3);
    prm.epoch = 1;
    prm.n_procs = r.p; prm.lanes = lanes; prm.slots = r.slots; prm.slot_elems = r.slot_elems;
    prm.blocking_send = r.blocking_send;
    if (dispatch(prm, r.dtype, r.op, r.wide, stream, false, nullptr) != cudaSuccess) return 1;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return 1;
    int status[2] = {0, 0};
    if (cudaMemcpy(status, base + oStatus, sizeof(status), cudaMemcpyDeviceToHost) != cudaSuccess) return 1;
    r.device_status = status[0];
    r.lanes = lanes;
    r.makespan_ns = 0.0;
    if (status[0] == 0 && r.h_block_times) {
        if (cudaMemcpy(r.h_block_times, base + oTimes, timeBytes, cudaMemcpyDeviceToHost) != cudaSuccess) return 1;
        unsigned long long begin = ~0ull, end = 0;
        for (size_t b = 0; b < size_t(r.p) * size_t(lanes); b++) if (r.h_block_times[2 * b] < begin) begin = r.h_block_times[2 * b];
        for (int g = 0; g < lanes; g++) if (r.h_block_times[2 * size_t(g) + 1] > end) end = r.h_block_times[2 * size_t(g) + 1];
        r.makespan_ns = end > begin ? double(end - begin) : 0.0;
    }
    return 0;
}

}  // namespace rd
