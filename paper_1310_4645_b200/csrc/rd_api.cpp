// The C ABI (see include/rd.h): argument checking, schedule objects, device tables, launches.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <vector>

#include "rd.h"
#include "rd_internal.h"
#include "rd_kernels.h"

using namespace rd;

namespace {

constexpr int kPtrRing = 8;   // pointer tables in flight for p > kPackedPtrs
constexpr int kMaxDevices = 64;

// Side streams of rd_reduce_batch, created on a device's first batch and kept for the process's life.
constexpr int kBatchRing = 4; // per-call tables of fused batches in flight
struct BatchLanes {
    bool ready = false;
    cudaStream_t stream[2] = {nullptr, nullptr};
    cudaEvent_t fork = nullptr, join[2] = {nullptr, nullptr};
    // fused batches: a pinned host ring and a device ring for the per-call tables (job descriptors,
    // per-CTA tile ranges, input pointer tables), one event per slot
    unsigned char *h_tab = nullptr, *d_tab = nullptr;
    size_t slot_bytes = 0;
    cudaEvent_t tab_done[kBatchRing] = {};
    bool tab_used[kBatchRing] = {};
    int tab_next = 0;
};
BatchLanes g_lanes[kMaxDevices];
std::mutex g_lanes_mutex;

// Counters for handing tiles out on demand (streaming kernel): a pool of word pairs per device, all zero
// between launches (the launch that used a pair zeroes it when its last CTA runs dry).  Launch k of the
// process on a device takes pair k mod kTileCounters, so a pair is shared only by launches that are 65536
// launches apart.  A launch that is being captured into a CUDA graph takes none (its CTAs work through fixed
// ranges): a replayed launch would otherwise keep using one pair beside whatever else is running.
constexpr uint32_t kTileCounters = 1u << 16;
struct TileCounters {
    uint32_t *pool = nullptr;
    bool failed = false;
    uint32_t next = 0;
};
TileCounters g_tile_counters[kMaxDevices];
std::mutex g_tile_counters_mutex;

uint32_t *next_tile_counter(int device, cudaStream_t stream)
{
    if (device < 0 || device >= kMaxDevices) return nullptr;
    if (stream) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) return nullptr;
    }
    std::lock_guard<std::mutex> hold(g_tile_counters_mutex);
    TileCounters &t = g_tile_counters[device];
    if (!t.pool && !t.failed) {
        const size_t bytes = size_t(kTileCounters) * 2 * sizeof(uint32_t);
        if (cudaMalloc(reinterpret_cast<void **>(&t.pool), bytes) != cudaSuccess || cudaMemset(t.pool, 0, bytes) != cudaSuccess) {
            cudaFree(t.pool);
            t.pool = nullptr;
            t.failed = true;
            (void)cudaGetLastError();
        }
    }
    if (!t.pool) return nullptr;
    uint32_t *pair = t.pool + 2u * size_t(t.next);
    t.next = (t.next + 1u) % kTileCounters;
    return pair;
}

// After a launch gave up a wait its pair may have been left non-zero: start again from a clean pool.
void reset_tile_counters(int device)
{
    if (device < 0 || device >= kMaxDevices) return;
    std::lock_guard<std::mutex> hold(g_tile_counters_mutex);
    TileCounters &t = g_tile_counters[device];
    if (t.pool) cudaMemset(t.pool, 0, size_t(kTileCounters) * 2 * sizeof(uint32_t));
}
constexpr int kDirectAutoProcs = 0;     // the direct kernel is never chosen by the library itself
constexpr int kTailTiles = 5; // key of the tile table for the elements the 128-bit path leaves over
constexpr int kPairTiles = 8; // key of the tile table of the 128-bit path with two operand tiles per ring stage
int tiles_key(int ops_per_stage) { return ops_per_stage == 2 ? kPairTiles : 4; }
// Levels the streaming kernel's shared-memory stack needs for a schedule's programs.
int ring_depth(const Programs &progs, int acc_words_per_word, int ops_per_stage)
{
    return stream_second_accumulator(acc_words_per_word, ops_per_stage) ? progs.shared_depth : progs.stack_depth;
}


struct DeviceTables {
    int device = -1;
    int sm_count = 0;
    int smem_per_sm = 0;
    uint32_t *ops = nullptr;
    std::map<int, std::pair<TileDesc *, uint32_t>> tiles;   // vector width -> (device table, count)
    // streaming (128-bit) path: tiles grouped per CTA, every CTA the same number of elements
    struct StreamPlan {                     // per-CTA tile ranges and ring shape of a single reduction's launch
        uint32_t *cta_first = nullptr;
        uint32_t n_ctas = 0;
        int ctas_per_sm = 0;
        int stages = 0;
    };
    std::map<int, StreamPlan> plans;        // key: 64 * (words of partial result per message word: 1, or 2 for 16-bit
                                            // elements) + 16 * operand tiles per ring stage + consumer warps
    int stage_elems = 0;
    int *status = nullptr;                                  // device word written by a kernel that gave up a wait
    // pointer tables for large p: pinned host ring + device ring, one event per slot
    void **h_ring = nullptr;
    void **d_ring = nullptr;
    cudaEvent_t ring_done[kPtrRing] = {};
    int ring_next = 0;
    cudaEvent_t ev_start = nullptr, ev_stop = nullptr;
    // schedule-faithful execution (allocated on its first use)
    bool faithful_ready = false;
    FaithfulAction *f_actions = nullptr;
    uint32_t *f_first = nullptr;
    uint64_t *f_seg_off = nullptr;
    uint32_t *f_flags = nullptr;            // posted, then taken: 2 * n_events * lanes words
    unsigned long long *f_trace = nullptr, *f_block_times = nullptr;
    uint32_t *f_scratch = nullptr;
    const uint32_t **f_inputs = nullptr;
    int *f_abort = nullptr;
    int f_lanes = 0, f_slots = 0;
    uint64_t f_slot_elems = 0;
    uint32_t f_epoch = 0;
    bool f_traced = false;
};

}  // namespace

struct rd_schedule {
    rd_algo_t algo;
    rd_port_t port;
    int p;
    size_t msg_bytes;
    rd_model_t model;
    Ticks ticks;
    std::vector<int64_t> seg_bytes;
    Schedule sched;
    Programs progs;
    double wait_budget_s = 2.0;             // bound of one wait inside the faithful kernel
    int tree_variant = RD_TREE_AUTO;        // which tree-mode kernel serves 16-byte aligned buffers
    DeviceTables dev;
};

namespace {

int make_ticks(const rd_model_t *m, Ticks &t)
{
    if (!m) return RD_ERR_INVALID_ARG;
    const double tick = m->tick > 0 ? m->tick : 1e-15;
    if (!(m->alpha >= 0) || !(m->beta >= 0) || !(m->gamma >= 0) || !std::isfinite(tick)) return RD_ERR_INVALID_ARG;
    const double a = m->alpha / tick, b = m->beta / tick, g = m->gamma / tick;
    if (!(a < 4e18) || !(b < 4e18) || !(g < 4e18)) return RD_ERR_INVALID_ARG;
    t.A = llround(a); t.B = llround(b); t.G = llround(g); t.tick = tick;
    // A communication must take time: with alpha and beta both zero (in ticks) every send of every schedule
    // starts and ends at time 0, the order of the events, and with it the combine order, is undefined.
    if (t.A == 0 && t.B == 0) return RD_ERR_INVALID_ARG;
    return RD_OK;
}

bool legal_pair(rd_algo_t algo, rd_port_t port)
{
    switch (algo) {
    case RD_UNI_GREEDY: return port == RD_PORT_UNI;
    case RD_BI_GREEDY: case RD_BUTTERFLY: return port == RD_PORT_BI;
    case RD_BINOMIAL: case RD_PIPELINE: case RD_BINARY: return port == RD_PORT_UNI || port == RD_PORT_BI;
    }
    return false;
}

int build(rd_schedule_t **out, rd_algo_t algo, rd_port_t port, int p, std::vector<int64_t> seg_bytes,
          size_t msg_bytes, const rd_model_t *model)
{
    if (!out || !model) return RD_ERR_INVALID_ARG;
    if (int(algo) < 0 || int(algo) > RD_BUTTERFLY || (port != RD_PORT_UNI && port != RD_PORT_BI)) return RD_ERR_INVALID_ARG;
    if (p < 1 || p > kMaxProcs) return RD_ERR_INVALID_ARG;
    if (!legal_pair(algo, port)) return RD_ERR_UNSUPPORTED;
    Ticks ticks;
    if (int rc = make_ticks(model, ticks)) return rc;
    // the largest time that can occur must stay far from int64 overflow
    {
        const long double worst = ((long double)ticks.A + ((long double)ticks.B + ticks.G) * (long double)msg_bytes) *
                                  ((long double)p + 2.0L * (long double)(seg_bytes.size() + 1)) * 4.0L;
        if (worst > 4.0e18L) return RD_ERR_INVALID_ARG;
    }
    rd_schedule *s = new (std::nothrow) rd_schedule();
    if (!s) return RD_ERR_NOMEM;
    int rc = RD_OK;
    try {
        s->algo = algo; s->port = port; s->p = p; s->msg_bytes = msg_bytes; s->model = *model; s->ticks = ticks;
        s->seg_bytes = std::move(seg_bytes);
        const bool bidir = port == RD_PORT_BI;
        switch (algo) {
        case RD_UNI_GREEDY: rc = gen_uni_greedy(p, s->seg_bytes, ticks, s->sched, true); break;
        case RD_BI_GREEDY: rc = gen_bi_greedy(p, s->seg_bytes, ticks, s->sched, true); break;
        case RD_BINOMIAL: rc = gen_binomial(p, s->seg_bytes, ticks, s->sched); break;
        case RD_PIPELINE: rc = gen_pipeline(p, s->seg_bytes, ticks, bidir, s->sched); break;
        case RD_BINARY: rc = gen_binary(p, s->seg_bytes, ticks, bidir, s->sched); break;
        case RD_BUTTERFLY: rc = gen_butterfly(p, msg_bytes / 4, ticks, s->sched); break;
        }
        if (rc == RD_OK) rc = compile_programs(p, s->sched.seg_off.size() - 1, s->sched.events, s->progs);
    } catch (const std::bad_alloc &) {
        rc = RD_ERR_NOMEM;
    }
    if (rc != RD_OK) { delete s; return rc; }
    *out = s;
    return RD_OK;
}

void release_device(DeviceTables &d)
{
    if (d.device < 0) return;
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(d.device);
    cudaFree(d.ops);
    for (auto &kv : d.plans) cudaFree(kv.second.cta_first);
    cudaFree(d.status);
    for (auto &kv : d.tiles) cudaFree(kv.second.first);
    if (d.h_ring) cudaFreeHost(d.h_ring);
    cudaFree(d.d_ring);
    for (auto &e : d.ring_done) if (e) cudaEventDestroy(e);
    if (d.ev_start) cudaEventDestroy(d.ev_start);
    if (d.ev_stop) cudaEventDestroy(d.ev_stop);
    cudaFree(d.f_actions); cudaFree(d.f_first); cudaFree(d.f_seg_off); cudaFree(d.f_flags); cudaFree(d.f_trace);
    cudaFree(d.f_block_times); cudaFree(d.f_scratch); cudaFree(d.f_inputs); cudaFree(d.f_abort);
    if (prev >= 0) cudaSetDevice(prev);
    d = DeviceTables();
}

int upload_tables(rd_schedule *s, int cur)
{
    DeviceTables &d = s->dev;
    d.device = cur;                          // from here on release_device frees whatever exists
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cur) != cudaSuccess) return RD_ERR_CUDA;
    d.sm_count = prop.multiProcessorCount;
    const size_t opBytes = std::max<size_t>(s->progs.ops.size(), 1) * sizeof(uint32_t);
    if (cudaMalloc(reinterpret_cast<void **>(&d.ops), opBytes) != cudaSuccess) return RD_ERR_NOMEM;
    if (!s->progs.ops.empty() &&
        cudaMemcpy(d.ops, s->progs.ops.data(), s->progs.ops.size() * sizeof(uint32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return RD_ERR_CUDA;
    if (cudaEventCreate(&d.ev_start) != cudaSuccess || cudaEventCreate(&d.ev_stop) != cudaSuccess) return RD_ERR_CUDA;
    if (cudaMalloc(reinterpret_cast<void **>(&d.status), sizeof(int)) != cudaSuccess) return RD_ERR_NOMEM;
    if (cudaMemset(d.status, 0, sizeof(int)) != cudaSuccess) return RD_ERR_CUDA;
    d.smem_per_sm = int(prop.sharedMemPerMultiprocessor);
    if (s->p > kPackedPtrs) {
        const size_t bytes = size_t(kPtrRing) * size_t(s->p) * sizeof(void *);
        if (cudaHostAlloc(reinterpret_cast<void **>(&d.h_ring), bytes, cudaHostAllocDefault) != cudaSuccess) return RD_ERR_NOMEM;
        if (cudaMalloc(reinterpret_cast<void **>(&d.d_ring), bytes) != cudaSuccess) return RD_ERR_NOMEM;
        for (auto &e : d.ring_done)
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return RD_ERR_CUDA;
    }
    return RD_OK;
}

// Copies the schedule's tables to the current device unless they are there already.  A failure
// half-way leaves nothing behind, so that the next call starts again from the beginning.
int upload(rd_schedule *s)
{
    DeviceTables &d = s->dev;
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) return RD_ERR_CUDA;
    if (d.device == cur) return RD_OK;
    if (d.device >= 0) release_device(d);
    const int rc = upload_tables(s, cur);
    if (rc != RD_OK) release_device(d);
    return rc;
}

// Tiles of the element-path kernel: runs of at most `cap` elements inside a segment.
int upload_tiles(DeviceTables &d, int key, const std::vector<TileDesc> &host)
{
    if (host.size() > 0xFFFFFFFFull) return RD_ERR_UNSUPPORTED;
    TileDesc *dev = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(&dev), std::max<size_t>(host.size(), 1) * sizeof(TileDesc)) != cudaSuccess)
        return RD_ERR_NOMEM;
    if (!host.empty() && cudaMemcpy(dev, host.data(), host.size() * sizeof(TileDesc), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaFree(dev);
        return RD_ERR_CUDA;
    }
    d.tiles.emplace(key, std::make_pair(dev, uint32_t(host.size())));
    return RD_OK;
}

int tiles_for(rd_schedule *s, int vec, const TileDesc **tiles, uint32_t *count)
{
    DeviceTables &d = s->dev;
    auto it = d.tiles.find(vec);
    if (it == d.tiles.end()) {
        const std::vector<uint64_t> &off = s->sched.seg_off;
        std::vector<TileDesc> host;
        if (vec == 4 || vec == kPairTiles) {
            // Streaming path.  Every segment is cut into equal tiles of at most one stage, or half a stage when
            // two operand tiles share a stage (whole 128-bit vectors of the buffers: where a segment starts or
            // ends inside a vector the tile is padded to the vector and remembers how many elements are not its own).
            const uint64_t n = off.empty() ? 0 : off.back();
            d.stage_elems = stream_stage_elems(n / (uint64_t(d.sm_count) * 2) + 1);
            const uint32_t cap = uint32_t(d.stage_elems) / (vec == kPairTiles ? 2u : 1u);
            const uint64_t n4 = n & ~uint64_t(3);          // the last n mod 4 elements go to the element kernel
            for (size_t seg = 0; seg + 1 < off.size(); seg++) {
                const uint64_t b = std::min(off[seg], n4), e = std::min(off[seg + 1], n4);
                if (e == b) continue;
                const uint64_t ps = b & ~uint64_t(3), pe = (e + 3) & ~uint64_t(3);
                const uint64_t parts = (pe - ps + cap - 1) / cap;
                const uint64_t each = std::min<uint64_t>(cap, ((pe - ps + parts - 1) / parts + 31) / 32 * 32);
                for (uint64_t ts = ps; ts < pe; ts += each) {
                    const uint64_t te = std::min<uint64_t>(pe, ts + each);
                    const uint32_t head = ts < b ? uint32_t(b - ts) : 0u, tail = te > e ? uint32_t(te - e) : 0u;
                    host.push_back(TileDesc{ts, uint32_t(te - ts) | (head << 16) | (tail << 18), s->progs.seg_prog[seg]});
                }
            }
        } else {
            // element path: the whole message (vec == 1), or only what the 128-bit path leaves over (kTailTiles)
            const uint64_t n = off.empty() ? 0 : off.back();
            const uint64_t from = vec == kTailTiles ? (n & ~uint64_t(3)) : 0;
            const uint32_t cap = tree_tile_elems(1);
            for (size_t j = 0; j + 1 < off.size(); j++)
                for (uint64_t e = std::max(off[j], from); e < off[j + 1]; e += cap)
                    host.push_back(TileDesc{e, uint32_t(std::min<uint64_t>(cap, off[j + 1] - e)), s->progs.seg_prog[j]});
        }
        if (int rc = upload_tiles(d, vec, host)) return rc;
        it = d.tiles.find(vec);
    }
    *tiles = it->second.first;
    *count = it->second.second;
    return RD_OK;
}

// Whether the schedule's programs push a partial result on the stack for at least every tenth operand (trees like
// the binomial one do for every fourth, the steady-state trees of uni-greedy for every fiftieth).
bool many_pushes(const rd_schedule *s)
{
    const size_t operands = size_t(s->p) * s->progs.seg_prog.size();
    return operands > 0 && s->progs.shared_pushes * 10 >= operands;
}

// Launch shape of a single reduction on the streaming path: CTAs get contiguous runs of tiles, the same
// NUMBER of tiles up to one (a tile costs a CTA about the same time however full it is, one ring hand-off
// per operation, so for small messages the number of tiles per CTA, not the number of elements, sets the
// kernel's duration; for large ones the two coincide).  acc_words: 2 for bf16, whose partial results are fp32.
int stream_plan(rd_schedule *s, int acc_words, int ops_per_stage, int consumer_warps, const DeviceTables::StreamPlan **out)
{
    DeviceTables &d = s->dev;
    const int key = 64 * acc_words + 16 * ops_per_stage + consumer_warps;
    auto it = d.plans.find(key);
    if (it == d.plans.end()) {
        const TileDesc *tiles = nullptr;
        uint32_t nTiles = 0;
        if (int rc = tiles_for(s, tiles_key(ops_per_stage), &tiles, &nTiles)) return rc;
        DeviceTables::StreamPlan plan;
        stream_shape(ring_depth(s->progs, acc_words, ops_per_stage), acc_words, ops_per_stage, many_pushes(s), d.smem_per_sm, d.stage_elems,
                     nTiles, d.sm_count, &plan.ctas_per_sm, &plan.stages);
        const uint64_t ctas = std::min<uint64_t>(uint64_t(d.sm_count) * uint64_t(plan.ctas_per_sm), std::max<uint64_t>(nTiles, 1));
        std::vector<uint32_t> first(size_t(ctas) + 1, 0);
        for (uint64_t c = 0; c < ctas; c++) first[size_t(c)] = uint32_t(uint64_t(nTiles) * c / ctas);
        first[size_t(ctas)] = nTiles;
        if (cudaMalloc(reinterpret_cast<void **>(&plan.cta_first), first.size() * sizeof(uint32_t)) != cudaSuccess) return RD_ERR_NOMEM;
        if (cudaMemcpy(plan.cta_first, first.data(), first.size() * sizeof(uint32_t), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(plan.cta_first);
            return RD_ERR_CUDA;
        }
        plan.n_ctas = uint32_t(ctas);
        it = d.plans.emplace(key, plan).first;
    }
    *out = &it->second;
    return RD_OK;
}

// Argument checks common to the reducing entry points.  On success *n_words is the message length
// in 32-bit words, the unit in which the schedule's segment boundaries and the kernels count.
bool is_half(rd_dtype_t dtype) { return dtype == RD_BF16 || dtype == RD_FP16; }
// Words of partial result per message word: the 16-bit types are widened to fp32 for sum and product; their
// max and min stay in 16 bits (the result of a combine is one of its operands).
int acc_words(rd_dtype_t dtype, rd_op_t op) { return is_half(dtype) && (op == RD_SUM || op == RD_PROD) ? 2 : 1; }
// Operand tiles per ring stage of the streaming kernel.  Where partial results are fp32 values of 16-bit elements
// a tile's waiting partial results take twice the shared memory of its operand: from stack depth 2 on such
// reductions run on tiles of half a stage, two to a stage (measured, bf16 sum, 64 MiB messages, GB/s, one tile
// against two tiles per stage: p = 2 6197 / 4705, p = 4 6616 / 6396, p = 8 6801 / 6838, p = 64 uni-greedy
// 6214 / 7174), unless the schedule asks for one kind of stage or the other.
int stage_ops(int acc_words_per_word, int tree_variant, int stack_depth)
{
    if (tree_variant == RD_TREE_STREAM) return 1;
    if (tree_variant == RD_TREE_STREAM_PAIRED) return 2;
    return acc_words_per_word > 1 && stack_depth >= 2 ? 2 : 1;
}
// Consumer warps of the streaming kernel: 8 with two vectors of a tile each, or 4 with four (two when two tiles
// share a stage).  Fewer warps with more vectors each spend fewer issue slots per byte, and with fewer instructions
// the SM clock settles higher under the board's power cap.  That pays for the 16-bit types, which have twice the
// elements per byte, for deep stacks, where shared memory leaves room for two thread blocks per SM only (measured,
// fp32 sum, p = 256, GB/s, 8 against 4 warps: binomial 6747 / 7104, uni-greedy 7109 / 7321), and from 16 processes
// on (p = 32, 1 GiB messages, a box whose SM clock is 1.6 GHz under the cap: uni- and bi-greedy, sum and max together
// 7092 / 7171, bi-greedy max 6882 / 7017; the batch of p = 64 with 4 MiB messages 7141 / 7172; at 1.85 GHz the two are
// level).  Fewer processes keep 8 warps: their launches are short, and a tile is finished sooner by more threads
// (p = 8, 64 KiB ... 1 MiB messages: 4 warps 4-5 % behind).
int stage_warps(int acc_words_per_word, int ops_per_stage, int stack_depth, int p)
{
    return ops_per_stage >= 2 || acc_words_per_word > 1 || stack_depth >= 6 || p >= 16 ? 4 : 8;
}
size_t elem_bytes(rd_dtype_t dtype) { return (dtype == RD_INT64 || dtype == RD_FP64) ? 8 : is_half(dtype) ? 2 : 4; }

int check_reduce_args(const rd_schedule *s, const void *const *d_inputs, const void *d_out, size_t n_elems, rd_dtype_t dtype,
                      rd_op_t op, size_t *n_words)
{
    if (!s || !d_inputs || int(dtype) < RD_INT32 || int(dtype) > RD_FP16 || int(op) < RD_SUM || int(op) > RD_PROD)
        return RD_ERR_INVALID_ARG;
    const size_t esize = elem_bytes(dtype);
    const size_t align = esize < 4 ? 4 : esize;          // the kernels move whole 32-bit words
    if (n_elems > s->msg_bytes / esize || n_elems * esize != s->msg_bytes) return RD_ERR_SIZE_MISMATCH;
    if (n_elems > 0 && !d_out) return RD_ERR_INVALID_ARG;
    for (int i = 0; i < s->p; i++)
        if ((n_elems > 0 && !d_inputs[i]) || (reinterpret_cast<uintptr_t>(d_inputs[i]) & (align - 1))) return RD_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_out) & (align - 1)) return RD_ERR_INVALID_ARG;
    if (esize == 8)                    // no segment may begin inside an element
        for (uint64_t off : s->sched.seg_off)
            if (off & 1u) return RD_ERR_INVALID_ARG;
    *n_words = s->msg_bytes / 4;
    return RD_OK;
}

int reduce_tree(rd_schedule *s, const void *const *d_inputs, void *d_out, size_t n, rd_dtype_t dtype, rd_op_t op,
                cudaStream_t stream, rd_stats_t *stats)
{
    DeviceTables &d = s->dev;
    // 128-bit path: every buffer 16-byte aligned (segments may start anywhere); the last n mod 4 elements
    // of the message, if any, are left to a second, tiny launch of the element kernel
    bool wide = (reinterpret_cast<uintptr_t>(d_out) & 15u) == 0;
    for (int i = 0; i < s->p && wide; i++) wide = (reinterpret_cast<uintptr_t>(d_inputs[i]) & 15u) == 0;
    TreeLaunch l{};
    l.vec = wide ? 4 : 1;
    l.ops_per_stage = stage_ops(acc_words(dtype, op), s->tree_variant, s->progs.shared_depth);
    l.consumer_warps = stage_warps(acc_words(dtype, op), l.ops_per_stage, s->progs.shared_depth, s->p);
    if (int rc = tiles_for(s, wide ? tiles_key(l.ops_per_stage) : 1, &l.tiles, &l.n_tiles)) return rc;
    const DeviceTables::StreamPlan *plan = nullptr;
    if (wide)
        if (int rc = stream_plan(s, acc_words(dtype, op), l.ops_per_stage, l.consumer_warps, &plan)) return rc;
    const TileDesc *tailTiles = nullptr;
    uint32_t nTail = 0;
    if (wide && (n & 3u) != 0)
        if (int rc = tiles_for(s, kTailTiles, &tailTiles, &nTail)) return rc;
    l.host_ptrs = d_inputs;
    l.dev_ptr_table = nullptr;
    if (s->p > kPackedPtrs) {
        const int slot = d.ring_next;
        d.ring_next = (d.ring_next + 1) % kPtrRing;
        if (cudaEventSynchronize(d.ring_done[slot]) != cudaSuccess) return RD_ERR_CUDA;   // previous user of the slot
        void **h = d.h_ring + size_t(slot) * size_t(s->p), **dv = d.d_ring + size_t(slot) * size_t(s->p);
        std::memcpy(h, d_inputs, size_t(s->p) * sizeof(void *));
        if (cudaMemcpyAsync(dv, h, size_t(s->p) * sizeof(void *), cudaMemcpyHostToDevice, stream) != cudaSuccess) return RD_ERR_CUDA;
        l.dev_ptr_table = dv;
    }
    l.out = d_out; l.ops = d.ops; l.p = s->p; l.stack_depth = s->progs.stack_depth;
    l.shared_depth = ring_depth(s->progs, acc_words(dtype, op), l.ops_per_stage);
    l.dtype = int(dtype); l.op = int(op); l.sm_count = d.sm_count; l.stream = stream;
    if (plan) { l.cta_first = plan->cta_first; l.n_ctas = plan->n_ctas; l.stages = plan->stages; }
    l.tile_counter = wide ? next_tile_counter(d.device, stream) : nullptr;
    l.stage_elems = d.stage_elems; l.status = d.status; l.device = d.device;
    // Direct kernel: all operands of an element in registers at once.  Only on request: since the streaming
    // kernel hands its tiles out on demand it is ahead for every process count (measured on B200, p = 2,
    // 1 GiB messages: 7.12 against 6.74 TB/s; p = 4: 7.24 against 6.94).
    const bool direct = wide && !is_half(dtype) && direct_applies(s->p, s->progs.stack_depth) &&
                        (s->tree_variant == RD_TREE_DIRECT || (s->tree_variant == RD_TREE_AUTO && s->p <= kDirectAutoProcs));
    if (stats && cudaEventRecord(d.ev_start, stream) != cudaSuccess) return RD_ERR_CUDA;
    if ((direct ? launch_tree_direct(l) : wide ? launch_tree_stream(l) : launch_tree(l)) != 0) return RD_ERR_CUDA;
    if (nTail > 0) {
        TreeLaunch t = l;
        t.vec = 1; t.tiles = tailTiles; t.n_tiles = nTail;
        if (launch_tree(t) != 0) return RD_ERR_CUDA;
    }
    if (s->p > kPackedPtrs) {
        const int slot = (d.ring_next + kPtrRing - 1) % kPtrRing;
        if (cudaEventRecord(d.ring_done[slot], stream) != cudaSuccess) return RD_ERR_CUDA;
    }
    if (stats) {
        if (cudaEventRecord(d.ev_stop, stream) != cudaSuccess) return RD_ERR_CUDA;
        if (cudaEventSynchronize(d.ev_stop) != cudaSuccess) return RD_ERR_CUDA;
        float ms = 0;
        if (cudaEventElapsedTime(&ms, d.ev_start, d.ev_stop) != cudaSuccess) return RD_ERR_CUDA;
        std::memset(stats, 0, sizeof(*stats));
        stats->kernel_ms = ms;
        stats->bytes_moved = uint64_t(s->p + 1) * uint64_t(n) * 4u;
        stats->gbytes_per_s = ms > 0 ? double(stats->bytes_moved) / (double(ms) * 1e6) : 0.0;
        stats->predicted_s = double(s->sched.completion) * s->ticks.tick;
        stats->n_launches = (l.n_tiles ? 1 : 0) + (nTail ? 1 : 0);
        int st = 0;
        if (cudaMemcpy(&st, d.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RD_ERR_CUDA;
        stats->device_status = st;
        if (st != 0) return RD_ERR_TIMEOUT;
    }
    return RD_OK;
}


template <typename T> int dev_alloc(T **ptr, size_t count)
{
    return cudaMalloc(reinterpret_cast<void **>(ptr), std::max<size_t>(count, 1) * sizeof(T)) == cudaSuccess ? RD_OK : RD_ERR_NOMEM;
}

// Words of one scratch slot: a segment that begins at word b of the message sits b mod 4 words into
// its slot (so that slot and messages agree on the 128-bit boundaries); whole vectors.
uint64_t faithful_slot_words(const std::vector<uint64_t> &seg_off)
{
    uint64_t need = 0;
    for (size_t j = 0; j + 1 < seg_off.size(); j++) need = std::max(need, (seg_off[j] & 3u) + (seg_off[j + 1] - seg_off[j]));
    return (need + 3) / 4 * 4;
}

// Device tables and scratch of the schedule-faithful execution, built on its first use.
int prepare_faithful(rd_schedule *s)
{
    DeviceTables &d = s->dev;
    if (d.faithful_ready) return RD_OK;
    // an earlier attempt may have failed half-way (out of memory): start clean
    cudaFree(d.f_actions); cudaFree(d.f_first); cudaFree(d.f_seg_off); cudaFree(d.f_flags); cudaFree(d.f_trace);
    cudaFree(d.f_block_times); cudaFree(d.f_scratch); cudaFree(d.f_inputs); cudaFree(d.f_abort);
    d.f_actions = nullptr; d.f_first = nullptr; d.f_seg_off = nullptr; d.f_flags = nullptr; d.f_trace = nullptr;
    d.f_block_times = nullptr; d.f_scratch = nullptr; d.f_inputs = nullptr; d.f_abort = nullptr;
    ActionLists lists;
    const size_t q = s->sched.seg_off.size() - 1;
    if (int rc = build_actions(s->p, q, s->sched.events, lists)) return rc;
    // all blocks have to be resident together: lanes per process from the least occupant variant
    int perSm = 1 << 30;
    for (int dt = 0; dt < 4; dt++)
        for (int op = 0; op < 4; op++)
            for (int wide = 0; wide < 2; wide++) {
                int b = 0;
                if (faithful_blocks_per_sm(dt, op, wide != 0, &b) != 0) return RD_ERR_CUDA;
                perSm = std::min(perSm, b);
            }
    const long long capacity = (long long)perSm * d.sm_count;
    if (capacity < s->p) return RD_ERR_UNSUPPORTED;
    d.f_lanes = int(std::min<long long>(16, capacity / s->p));
    d.f_slots = std::max(lists.slots_per_proc, 1);
    d.f_slot_elems = faithful_slot_words(s->sched.seg_off);
    const size_t nEvents = s->sched.events.size();
    std::vector<FaithfulAction> acts(lists.actions.size());
    for (size_t k = 0; k < acts.size(); k++) {
        const Action &a = lists.actions[k];
        acts[k] = FaithfulAction{a.seg, a.peer, a.kind, a.slot, a.peer_slot, a.first, a.event, a.wait_event};
    }
    if (dev_alloc(&d.f_actions, acts.size()) || dev_alloc(&d.f_first, lists.first.size()) ||
        dev_alloc(&d.f_seg_off, s->sched.seg_off.size()) || dev_alloc(&d.f_flags, 2 * nEvents * size_t(d.f_lanes)) ||
        dev_alloc(&d.f_trace, 3 * nEvents) || dev_alloc(&d.f_block_times, 2 * size_t(s->p) * size_t(d.f_lanes)) ||
        dev_alloc(&d.f_inputs, size_t(s->p)) || dev_alloc(&d.f_abort, 1) ||
        dev_alloc(&d.f_scratch, size_t(s->p) * size_t(d.f_slots) * size_t(d.f_slot_elems)))
        return RD_ERR_NOMEM;
    bool ok = true;
    ok = ok && (acts.empty() || cudaMemcpy(d.f_actions, acts.data(), acts.size() * sizeof(FaithfulAction), cudaMemcpyHostToDevice) == cudaSuccess);
    ok = ok && cudaMemcpy(d.f_first, lists.first.data(), lists.first.size() * sizeof(uint32_t), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(d.f_seg_off, s->sched.seg_off.data(), s->sched.seg_off.size() * sizeof(uint64_t), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemset(d.f_flags, 0, std::max<size_t>(2 * nEvents * size_t(d.f_lanes), 1) * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMemset(d.f_trace, 0, std::max<size_t>(3 * nEvents, 1) * sizeof(unsigned long long)) == cudaSuccess;
    ok = ok && cudaMemset(d.f_abort, 0, sizeof(int)) == cudaSuccess;
    if (!ok) return RD_ERR_CUDA;
    d.f_epoch = 0;
    d.faithful_ready = true;
    return RD_OK;
}

int reduce_faithful(rd_schedule *s, const void *const *d_inputs, void *d_out, size_t n, rd_dtype_t dtype, rd_op_t op,
                    cudaStream_t stream, rd_stats_t *stats)
{
    DeviceTables &d = s->dev;
    rd_stats_t st;
    std::memset(&st, 0, sizeof(st));
    st.bytes_moved = uint64_t(s->p + 1) * uint64_t(n) * 4u;
    st.predicted_s = double(s->sched.completion) * s->ticks.tick;
    if (n == 0) { if (stats) *stats = st; return RD_OK; }
    if (cudaEventRecord(d.ev_start, stream) != cudaSuccess) return RD_ERR_CUDA;
    if (s->p == 1) {
        // a single process holds the result already
        if (d_out != d_inputs[0] && cudaMemcpyAsync(d_out, d_inputs[0], n * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
            return RD_ERR_CUDA;
    } else {
        if (int rc = prepare_faithful(s)) return rc;
        bool wide = (reinterpret_cast<uintptr_t>(d_out) & 15u) == 0;
        for (int i = 0; i < s->p && wide; i++) wide = (reinterpret_cast<uintptr_t>(d_inputs[i]) & 15u) == 0;
        if (cudaMemcpyAsync(d.f_inputs, d_inputs, size_t(s->p) * sizeof(void *), cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return RD_ERR_CUDA;
        if (++d.f_epoch == 0) d.f_epoch = 1;
        const size_t nEvents = s->sched.events.size();
        FaithfulParams prm{};
        prm.inputs = reinterpret_cast<const uint32_t *const *>(d.f_inputs);
        prm.out = static_cast<uint32_t *>(d_out);
        prm.scratch = d.f_scratch; prm.actions = d.f_actions; prm.first = d.f_first; prm.seg_off = d.f_seg_off;
        prm.posted = d.f_flags; prm.taken = d.f_flags + nEvents * size_t(d.f_lanes);
        prm.trace = d.f_trace; prm.block_times = d.f_block_times; prm.status = d.status; prm.abort_flag = d.f_abort;
        int khz = 0;
        cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, d.device);
        prm.wait_cycles = (long long)(s->wait_budget_s * double(khz > 0 ? khz : 1000000) * 1e3);
        prm.epoch = d.f_epoch; prm.n_procs = s->p; prm.lanes = d.f_lanes; prm.slots = d.f_slots;
        prm.slot_elems = d.f_slot_elems; prm.blocking_send = s->port == RD_PORT_UNI ? 1 : 0;
        if (launch_faithful(prm, int(dtype), int(op), wide, stream) != 0) return RD_ERR_CUDA;
        st.n_launches = 1;
        d.f_traced = true;
    }
    if (cudaEventRecord(d.ev_stop, stream) != cudaSuccess || cudaEventSynchronize(d.ev_stop) != cudaSuccess) return RD_ERR_CUDA;
    float ms = 0;
    if (cudaEventElapsedTime(&ms, d.ev_start, d.ev_stop) != cudaSuccess) return RD_ERR_CUDA;
    st.kernel_ms = ms;
    st.gbytes_per_s = ms > 0 ? double(st.bytes_moved) / (double(ms) * 1e6) : 0.0;
    if (s->p > 1) {
        int status = 0;
        if (cudaMemcpy(&status, d.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RD_ERR_CUDA;
        st.device_status = status;
        if (status != 0) {
            // leave the flags usable for the next call: new epoch, cleared status and abort flag
            cudaMemset(d.status, 0, sizeof(int));
            cudaMemset(d.f_abort, 0, sizeof(int));
            if (stats) *stats = st;
            return RD_ERR_TIMEOUT;
        }
        std::vector<unsigned long long> bt(2 * size_t(s->p) * size_t(d.f_lanes));
        if (cudaMemcpy(bt.data(), d.f_block_times, bt.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess)
            return RD_ERR_CUDA;
        unsigned long long begin = ~0ull, end = 0;
        for (size_t b = 0; b < bt.size() / 2; b++) begin = std::min(begin, bt[2 * b]);
        for (int g = 0; g < d.f_lanes; g++) end = std::max(end, bt[2 * size_t(g) + 1]);     // the root's blocks
        st.makespan_ns = end > begin ? double(end - begin) : 0.0;
    }
    if (stats) *stats = st;
    return RD_OK;
}

// A batch as ONE launch of the streaming kernel: the tiles of all jobs are numbered through and dealt
// to the thread blocks like the tiles of a single reduction, so the launch has one fill and one tail and
// the ring shape is chosen for the batch's total number of tiles.  The job descriptors and the jobs' input
// pointers travel as kernel parameters when they fit, else in one copy from a pinned ring.
int reduce_batch_fused(size_t n_jobs, rd_schedule_t *const *schedules, const void *const *const *d_inputs, void *const *d_outs,
                       rd_dtype_t dtype, rd_op_t op, cudaStream_t user)
{
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return RD_ERR_CUDA;
    std::vector<BatchJob> jobs(n_jobs);
    uint64_t total = 0;
    size_t nPtrs = 0;
    int depth = 0;
    for (size_t j = 0; j < n_jobs; j++) depth = std::max(depth, schedules[j]->progs.shared_depth);
    const int opsPerStage = stage_ops(acc_words(dtype, op), RD_TREE_AUTO, depth);  // one kind of stage for the whole launch
    if (!stream_second_accumulator(acc_words(dtype, op), opsPerStage))             // levels in shared memory
        for (size_t j = 0; j < n_jobs; j++) depth = std::max(depth, schedules[j]->progs.stack_depth);
    for (size_t j = 0; j < n_jobs; j++) {
        rd_schedule *s = schedules[j];
        const TileDesc *tiles = nullptr;
        uint32_t count = 0;
        if (int rc = tiles_for(s, tiles_key(opsPerStage), &tiles, &count)) return rc;
        BatchJob &b = jobs[j];
        b.inputs = nullptr; b.out = static_cast<uint32_t *>(d_outs[j]); b.tiles = tiles; b.ops = s->dev.ops;
        b.tile_begin = uint32_t(total); b.p = s->p; b.ptr_base = 0;
        total += count;
        if (total > 0xFFFFFFFFull) return RD_ERR_UNSUPPORTED;
        b.tile_end = uint32_t(total);
        nPtrs += size_t(s->p);
    }
    if (total == 0) return RD_OK;
    DeviceTables &d0 = schedules[0]->dev;
    const int stageElems = d0.stage_elems;
    int ctasPerSm = 1, stages = 2;
    int mostProcs = 0;
    for (size_t j = 0; j < n_jobs; j++) mostProcs = std::max(mostProcs, schedules[j]->p);
    const int consumerWarps = stage_warps(acc_words(dtype, op), opsPerStage, depth, mostProcs);
    bool pushy = false;
    for (size_t j = 0; j < n_jobs; j++) pushy = pushy || many_pushes(schedules[j]);
    stream_shape(depth, acc_words(dtype, op), opsPerStage, pushy, d0.smem_per_sm, stageElems, total, d0.sm_count, &ctasPerSm, &stages);
    const uint64_t ctas = std::min<uint64_t>(uint64_t(d0.sm_count) * uint64_t(ctasPerSm), total);
    BatchLaunch b{};
    b.n_jobs = uint32_t(n_jobs); b.n_tiles = uint32_t(total); b.n_ctas = uint32_t(ctas);
    b.stages = stages; b.stack_depth = depth; b.stage_elems = stageElems; b.ops_per_stage = opsPerStage; b.consumer_warps = consumerWarps;
    b.dtype = int(dtype); b.op = int(op); b.device = device; b.status = d0.status; b.stream = user;
    b.tile_counter = next_tile_counter(device, user);
    if (n_jobs <= size_t(kBatchPackJobs) && nPtrs <= size_t(kBatchPackPtrs)) {
        // small batch: descriptors and pointers travel as kernel parameters, nothing is copied ahead of the launch
        std::vector<const void *> ptrs(nPtrs);
        size_t at = 0;
        for (size_t j = 0; j < n_jobs; j++) {
            jobs[j].ptr_base = int(at);
            for (int i = 0; i < schedules[j]->p; i++) ptrs[at++] = d_inputs[j][i];
        }
        b.host_jobs = jobs.data(); b.host_ptrs = ptrs.data(); b.n_ptrs = uint32_t(nPtrs);
        return launch_tree_stream_batch(b) == 0 ? RD_OK : RD_ERR_CUDA;
    }
    // layout of a slot of the ring: job descriptors | input pointers of all jobs
    const size_t oPtrs = (n_jobs * sizeof(BatchJob) + 15) & ~size_t(15);
    const size_t need = oPtrs + nPtrs * sizeof(void *);

    std::lock_guard<std::mutex> hold(g_lanes_mutex);
    BatchLanes &lanes = g_lanes[device];
    if (need > lanes.slot_bytes) {
        // grow: wait for the launches that still read the old ring, then replace it
        for (int k = 0; k < kBatchRing; k++)
            if (lanes.tab_used[k] && cudaEventSynchronize(lanes.tab_done[k]) != cudaSuccess) return RD_ERR_CUDA;
        if (lanes.h_tab) cudaFreeHost(lanes.h_tab);
        cudaFree(lanes.d_tab);
        lanes.h_tab = lanes.d_tab = nullptr;
        lanes.slot_bytes = 0;
        size_t slot = 64 << 10;
        while (slot < need) slot *= 2;
        if (cudaHostAlloc(reinterpret_cast<void **>(&lanes.h_tab), slot * kBatchRing, cudaHostAllocDefault) != cudaSuccess) return RD_ERR_NOMEM;
        if (cudaMalloc(reinterpret_cast<void **>(&lanes.d_tab), slot * kBatchRing) != cudaSuccess) {
            cudaFreeHost(lanes.h_tab);
            lanes.h_tab = nullptr;
            return RD_ERR_NOMEM;
        }
        for (int k = 0; k < kBatchRing; k++) {
            if (!lanes.tab_done[k] && cudaEventCreateWithFlags(&lanes.tab_done[k], cudaEventDisableTiming) != cudaSuccess) return RD_ERR_CUDA;
            lanes.tab_used[k] = false;
        }
        lanes.slot_bytes = slot;
    }
    const int slot = lanes.tab_next;
    lanes.tab_next = (lanes.tab_next + 1) % kBatchRing;
    if (lanes.tab_used[slot] && cudaEventSynchronize(lanes.tab_done[slot]) != cudaSuccess) return RD_ERR_CUDA;   // the slot's previous launch
    unsigned char *h = lanes.h_tab + size_t(slot) * lanes.slot_bytes, *dv = lanes.d_tab + size_t(slot) * lanes.slot_bytes;
    const void **hp = reinterpret_cast<const void **>(h + oPtrs);
    size_t at = 0;
    for (size_t j = 0; j < n_jobs; j++) {
        jobs[j].inputs = reinterpret_cast<const uint32_t *const *>(dv + oPtrs) + at;
        for (int i = 0; i < schedules[j]->p; i++) hp[at++] = d_inputs[j][i];
    }
    std::memcpy(h, jobs.data(), n_jobs * sizeof(BatchJob));
    if (cudaMemcpyAsync(dv, h, need, cudaMemcpyHostToDevice, user) != cudaSuccess) return RD_ERR_CUDA;
    b.jobs = reinterpret_cast<const BatchJob *>(dv);
    const int launched = launch_tree_stream_batch(b);
    lanes.tab_used[slot] = cudaEventRecord(lanes.tab_done[slot], user) == cudaSuccess;
    if (launched != 0 || !lanes.tab_used[slot]) return RD_ERR_CUDA;
    return RD_OK;
}

// Nothing may be thrown across the C boundary: host containers can run out of memory.
template <typename F> int guarded(F &&body)
{
    try {
        return body();
    } catch (const std::bad_alloc &) {
        return RD_ERR_NOMEM;
    } catch (...) {
        return RD_ERR_INTERNAL;
    }
}

}  // namespace

extern "C" {

int rd_schedule_create(rd_schedule_t **out, rd_algo_t algo, rd_port_t port, int p, size_t msg_bytes, size_t seg_bytes,
                       const rd_model_t *model)
{
    if (!out || !model || (msg_bytes & 3u) || (seg_bytes & 3u)) return RD_ERR_INVALID_ARG;
    if (p < 1 || p > kMaxProcs) return RD_ERR_INVALID_ARG;
    if (int(algo) < 0 || int(algo) > RD_BUTTERFLY || (port != RD_PORT_UNI && port != RD_PORT_BI)) return RD_ERR_INVALID_ARG;
    if (!legal_pair(algo, port)) return RD_ERR_UNSUPPORTED;
    if (seg_bytes == 0) {
        Ticks t;
        if (int rc = make_ticks(model, t)) return rc;
        if (int rc = optimal_segment(algo, port, p, msg_bytes, t, &seg_bytes)) return rc;
    }
    std::vector<int64_t> segs;
    try {
        if (algo != RD_BUTTERFLY) {
            if (seg_bytes > msg_bytes) seg_bytes = msg_bytes;
            if (msg_bytes > 0 && (msg_bytes + seg_bytes - 1) / seg_bytes > (size_t(1) << 22)) return RD_ERR_INVALID_ARG;
            for (size_t done = 0; done < msg_bytes; done += seg_bytes)
                segs.push_back(int64_t(std::min(seg_bytes, msg_bytes - done)));
        }
    } catch (const std::bad_alloc &) {
        return RD_ERR_NOMEM;
    }
    return build(out, algo, port, p, std::move(segs), msg_bytes, model);
}

int rd_schedule_create_segments(rd_schedule_t **out, rd_algo_t algo, rd_port_t port, int p, const size_t *seg_bytes,
                                size_t q, const rd_model_t *model)
{
    if (!out || !model || (!seg_bytes && q > 0)) return RD_ERR_INVALID_ARG;
    if (algo == RD_BUTTERFLY) return RD_ERR_UNSUPPORTED;
    if (q > (size_t(1) << 22)) return RD_ERR_INVALID_ARG;
    std::vector<int64_t> segs;
    size_t total = 0;
    try {
        for (size_t j = 0; j < q; j++) {
            if (seg_bytes[j] == 0 || (seg_bytes[j] & 3u)) return RD_ERR_INVALID_ARG;
            segs.push_back(int64_t(seg_bytes[j]));
            total += seg_bytes[j];
        }
    } catch (const std::bad_alloc &) {
        return RD_ERR_NOMEM;
    }
    return build(out, algo, port, p, std::move(segs), total, model);
}

int rd_optimal_segment(rd_algo_t algo, rd_port_t port, int p, size_t msg_bytes, const rd_model_t *model, size_t *seg_bytes_out)
{
    if (!model || !seg_bytes_out || (msg_bytes & 3u) || p < 1 || p > kMaxProcs) return RD_ERR_INVALID_ARG;
    if (int(algo) < 0 || int(algo) > RD_BUTTERFLY || (port != RD_PORT_UNI && port != RD_PORT_BI)) return RD_ERR_INVALID_ARG;
    if (!legal_pair(algo, port)) return RD_ERR_UNSUPPORTED;
    Ticks t;
    if (int rc = make_ticks(model, t)) return rc;
    size_t s = 0;
    try {
        if (int rc = optimal_segment(algo, port, p, msg_bytes, t, &s)) return rc;
    } catch (const std::bad_alloc &) {
        return RD_ERR_NOMEM;
    }
    *seg_bytes_out = s;
    return RD_OK;
}

int rd_schedule_info(const rd_schedule_t *s, int *p, size_t *q, size_t *n_events, double *predicted_seconds,
                     int64_t *predicted_ticks, int *stack_depth)
{
    if (!s) return RD_ERR_INVALID_ARG;
    if (p) *p = s->p;
    if (q) *q = s->sched.seg_off.size() - 1;
    if (n_events) *n_events = s->sched.events.size();
    if (predicted_seconds) *predicted_seconds = double(s->sched.completion) * s->ticks.tick;
    if (predicted_ticks) *predicted_ticks = s->sched.completion;
    if (stack_depth) *stack_depth = s->progs.stack_depth;
    return RD_OK;
}

int rd_schedule_events(const rd_schedule_t *s, rd_event_t *buf, size_t cap)
{
    if (!s || (!buf && cap > 0)) return RD_ERR_INVALID_ARG;
    if (cap < s->sched.events.size()) return RD_ERR_TOO_SMALL;
    if (!s->sched.events.empty()) std::memcpy(buf, s->sched.events.data(), s->sched.events.size() * sizeof(rd_event_t));
    return RD_OK;
}

int rd_schedule_segments(const rd_schedule_t *s, uint64_t *off, size_t cap)
{
    if (!s || !off) return RD_ERR_INVALID_ARG;
    if (cap < s->sched.seg_off.size()) return RD_ERR_TOO_SMALL;
    std::memcpy(off, s->sched.seg_off.data(), s->sched.seg_off.size() * sizeof(uint64_t));
    return RD_OK;
}

int rd_schedule_program(const rd_schedule_t *s, size_t seg, uint32_t *ops, size_t cap)
{
    if (!s || !ops || seg >= s->progs.seg_prog.size()) return RD_ERR_INVALID_ARG;
    if (cap < size_t(s->p)) return RD_ERR_TOO_SMALL;
    std::memcpy(ops, s->progs.ops.data() + s->progs.seg_prog[seg], size_t(s->p) * sizeof(uint32_t));
    return RD_OK;
}

int rd_schedule_upload(rd_schedule_t *s)
{
    if (!s) return RD_ERR_INVALID_ARG;
    return guarded([&] { return upload(s); });
}

int rd_reduce(rd_schedule_t *s, const void *const *d_inputs, void *d_out, size_t n_elems, rd_dtype_t dtype, rd_op_t op,
              rd_exec_t exec, void *cuda_stream, rd_stats_t *stats)
{
    if (exec != RD_EXEC_TREE && exec != RD_EXEC_FAITHFUL) return RD_ERR_INVALID_ARG;
    size_t n_words = 0;
    if (int rc = check_reduce_args(s, d_inputs, d_out, n_elems, dtype, op, &n_words)) return rc;
    if (exec == RD_EXEC_FAITHFUL && is_half(dtype)) return RD_ERR_UNSUPPORTED;   // partial segments would be fp32
    return guarded([&] {
        if (int rc = upload(s)) return rc;
        if (exec == RD_EXEC_FAITHFUL)
            return reduce_faithful(s, d_inputs, d_out, n_words, dtype, op, static_cast<cudaStream_t>(cuda_stream), stats);
        return reduce_tree(s, d_inputs, d_out, n_words, dtype, op, static_cast<cudaStream_t>(cuda_stream), stats);
    });
}

int rd_allreduce(rd_schedule_t *s, const void *const *d_inputs, void *const *d_outs, size_t n_elems, rd_dtype_t dtype, rd_op_t op,
                 void *cuda_stream, rd_stats_t *stats)
{
    if (!s || !d_outs) return RD_ERR_INVALID_ARG;
    size_t n_words = 0;
    if (int rc = check_reduce_args(s, d_inputs, d_outs[0], n_elems, dtype, op, &n_words)) return rc;
    const size_t bytes = n_words * 4;
    const size_t align = elem_bytes(dtype) < 4 ? 4 : elem_bytes(dtype);
    auto overlap = [bytes](const void *a, const void *b) {
        const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
        return bytes > 0 && x < y + bytes && y < x + bytes;
    };
    bool wide = true;                                  // every copy 16-byte aligned
    for (int i = 0; i < s->p; i++) {
        if ((n_elems > 0 && !d_outs[i]) || (reinterpret_cast<uintptr_t>(d_outs[i]) & (align - 1))) return RD_ERR_INVALID_ARG;
        wide = wide && (reinterpret_cast<uintptr_t>(d_outs[i]) & 15u) == 0;
        // the copies are written while other processes' inputs may still be read: a copy may only coincide with
        // its own process's input (the in-place all-reduce), and no two copies may overlap
        for (int k = 0; k < s->p; k++) {
            if (k != i && overlap(d_outs[i], d_inputs[k])) return RD_ERR_INVALID_ARG;
            if (k > i && overlap(d_outs[i], d_outs[k])) return RD_ERR_INVALID_ARG;
        }
        if (d_outs[i] != d_inputs[i] && overlap(d_outs[i], d_inputs[i])) return RD_ERR_INVALID_ARG;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    return guarded([&]() -> int {
        if (int rc = upload(s)) return rc;
        DeviceTables &d = s->dev;
        if (stats && cudaEventRecord(d.ev_start, stream) != cudaSuccess) return RD_ERR_CUDA;
        // Section III: a reduce to the root followed by a broadcast of the root's result
        if (int rc = reduce_tree(s, d_inputs, d_outs[0], n_words, dtype, op, stream, nullptr)) return rc;
        if (s->p > 1 && launch_broadcast(d_outs[0], d_outs + 1, s->p - 1, n_words, wide, d.sm_count, d.status, stream) != 0) return RD_ERR_CUDA;
        if (stats) {
            if (cudaEventRecord(d.ev_stop, stream) != cudaSuccess || cudaEventSynchronize(d.ev_stop) != cudaSuccess) return RD_ERR_CUDA;
            float ms = 0;
            if (cudaEventElapsedTime(&ms, d.ev_start, d.ev_stop) != cudaSuccess) return RD_ERR_CUDA;
            std::memset(stats, 0, sizeof(*stats));
            stats->kernel_ms = ms;
            stats->bytes_moved = (uint64_t(s->p + 1) + uint64_t(s->p > 1 ? s->p : 0)) * uint64_t(bytes);
            stats->gbytes_per_s = ms > 0 ? double(stats->bytes_moved) / (double(ms) * 1e6) : 0.0;
            stats->predicted_s = double(s->sched.completion) * s->ticks.tick;
            bool vectors = (reinterpret_cast<uintptr_t>(d_outs[0]) & 15u) == 0;      // the reduction took the 128-bit path
            for (int i = 0; i < s->p && vectors; i++) vectors = (reinterpret_cast<uintptr_t>(d_inputs[i]) & 15u) == 0;
            stats->n_launches = n_words ? 1 + (vectors && (n_words & 3u) ? 1 : 0) + broadcast_launches(s->p - 1, n_words, wide) : 0;
            int st = 0;
            if (cudaMemcpy(&st, d.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RD_ERR_CUDA;
            stats->device_status = st;
            if (st != 0) return RD_ERR_TIMEOUT;
        }
        return RD_OK;
    });
}

int rd_reduce_batch(size_t n_jobs, rd_schedule_t *const *schedules, const void *const *const *d_inputs, void *const *d_outs,
                    const size_t *n_elems, rd_dtype_t dtype, rd_op_t op, void *cuda_stream)
{
    if (n_jobs == 0) return RD_OK;
    if (!schedules || !d_inputs || !d_outs || !n_elems) return RD_ERR_INVALID_ARG;
    std::vector<size_t> words;
    try { words.resize(n_jobs); } catch (const std::bad_alloc &) { return RD_ERR_NOMEM; }
    for (size_t j = 0; j < n_jobs; j++) {
        if (!schedules[j] || !d_inputs[j]) return RD_ERR_INVALID_ARG;
        if (int rc = check_reduce_args(schedules[j], d_inputs[j], d_outs[j], n_elems[j], dtype, op, &words[j])) return rc;
    }
    // the jobs may run concurrently: no job's output may overlap another job's output or inputs
    // (a job's own output may alias its own root input, as in rd_reduce)
    auto overlap = [](const void *a, size_t na, const void *b, size_t nb) {
        const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
        return na > 0 && nb > 0 && x < y + nb && y < x + na;
    };
    for (size_t j = 0; j < n_jobs; j++)
        for (size_t k = 0; k < n_jobs; k++) {
            if (k == j) continue;
            if (k > j && overlap(d_outs[j], words[j] * 4, d_outs[k], words[k] * 4)) return RD_ERR_INVALID_ARG;
            for (int i = 0; i < schedules[k]->p; i++)
                if (overlap(d_outs[j], words[j] * 4, d_inputs[k][i], words[k] * 4)) return RD_ERR_INVALID_ARG;
        }
    cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
    return guarded([&] {
        for (size_t j = 0; j < n_jobs; j++)
            if (int rc = upload(schedules[j])) return rc;
        if (n_jobs == 1) return reduce_tree(schedules[0], d_inputs[0], d_outs[0], words[0], dtype, op, user, nullptr);
        // One launch for the whole batch when every job can take the 128-bit streaming path by itself
        // (all buffers 16-byte aligned, whole vectors).
        bool fuse = true;
        for (size_t j = 0; j < n_jobs && fuse; j++) {
            fuse = (words[j] & 3u) == 0 && (reinterpret_cast<uintptr_t>(d_outs[j]) & 15u) == 0;
            for (int i = 0; i < schedules[j]->p && fuse; i++) fuse = (reinterpret_cast<uintptr_t>(d_inputs[j][i]) & 15u) == 0;
        }
        if (fuse) {
            const int rc = reduce_batch_fused(n_jobs, schedules, d_inputs, d_outs, dtype, op, user);
            if (rc != RD_ERR_UNSUPPORTED) return rc;        // UNSUPPORTED: more tiles than one launch can number
        }
        // Fork: two side streams wait for what precedes the batch on the caller's stream and take the
        // jobs alternately, so that one job's thread blocks fill the SM slots the other job frees while
        // its last blocks are still running.  Join: the caller's stream waits for both.
        int device = -1;
        if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return int(RD_ERR_CUDA);
        std::lock_guard<std::mutex> hold(g_lanes_mutex);
        BatchLanes &lanes = g_lanes[device];
        if (!lanes.ready) {
            bool ok = cudaEventCreateWithFlags(&lanes.fork, cudaEventDisableTiming) == cudaSuccess;
            for (int l = 0; l < 2 && ok; l++)
                ok = cudaStreamCreateWithFlags(&lanes.stream[l], cudaStreamNonBlocking) == cudaSuccess &&
                     cudaEventCreateWithFlags(&lanes.join[l], cudaEventDisableTiming) == cudaSuccess;
            if (!ok) return int(RD_ERR_CUDA);
            lanes.ready = true;
        }
        if (cudaEventRecord(lanes.fork, user) != cudaSuccess) return int(RD_ERR_CUDA);
        for (int l = 0; l < 2; l++)
            if (cudaStreamWaitEvent(lanes.stream[l], lanes.fork, 0) != cudaSuccess) return int(RD_ERR_CUDA);
        int rc = RD_OK;
        for (size_t j = 0; j < n_jobs && rc == RD_OK; j++)
            rc = reduce_tree(schedules[j], d_inputs[j], d_outs[j], words[j], dtype, op, lanes.stream[j & 1], nullptr);
        // join also after a failure, so that what was launched stays ordered before the caller's next work
        for (int l = 0; l < 2; l++)
            if (cudaEventRecord(lanes.join[l], lanes.stream[l]) != cudaSuccess || cudaStreamWaitEvent(user, lanes.join[l], 0) != cudaSuccess)
                rc = rc == RD_OK ? int(RD_ERR_CUDA) : rc;
        return rc;
    });
}

int rd_reduce_host(rd_schedule_t *s, const void *const *h_inputs, void *h_out, void *d_staging, size_t n_elems,
                   rd_dtype_t dtype, rd_op_t op, void *cuda_stream)
{
    if (!s || !h_inputs || (n_elems > 0 && (!h_out || !d_staging))) return RD_ERR_INVALID_ARG;
    if (int(dtype) < RD_INT32 || int(dtype) > RD_FP16) return RD_ERR_INVALID_ARG;
    if (n_elems > s->msg_bytes / elem_bytes(dtype) || n_elems * elem_bytes(dtype) != s->msg_bytes) return RD_ERR_SIZE_MISMATCH;
    const size_t row = s->msg_bytes;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    std::vector<const void *> dptr;
    try { dptr.resize(size_t(s->p)); } catch (const std::bad_alloc &) { return RD_ERR_NOMEM; }
    char *base = static_cast<char *>(d_staging);
    for (int i = 0; i < s->p; i++) {
        if (n_elems > 0 && !h_inputs[i]) return RD_ERR_INVALID_ARG;
        dptr[size_t(i)] = base + size_t(i) * row;
    }
    // messages that follow each other in host memory (the rows of one array) travel in one copy
    for (int i = 0; i < s->p && n_elems > 0;) {
        int j = i + 1;
        while (j < s->p && static_cast<const char *>(h_inputs[j]) == static_cast<const char *>(h_inputs[j - 1]) + row) j++;
        if (cudaMemcpyAsync(base + size_t(i) * row, h_inputs[i], size_t(j - i) * row, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return RD_ERR_CUDA;
        i = j;
    }
    void *d_out = base + size_t(s->p) * row;
    if (int rc = rd_reduce(s, dptr.data(), d_out, n_elems, dtype, op, RD_EXEC_TREE, cuda_stream, nullptr)) return rc;
    if (n_elems > 0 && cudaMemcpyAsync(h_out, d_out, row, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return RD_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return RD_ERR_CUDA;
    return RD_OK;
}

int rd_schedule_set_wait_budget(rd_schedule_t *s, double seconds)
{
    if (!s || !(seconds > 0) || !(seconds <= 60.0)) return RD_ERR_INVALID_ARG;
    s->wait_budget_s = seconds;
    return RD_OK;
}

int rd_schedule_set_tree_variant(rd_schedule_t *s, rd_tree_variant_t variant)
{
    if (!s || int(variant) < RD_TREE_AUTO || int(variant) > RD_TREE_STREAM_PAIRED) return RD_ERR_INVALID_ARG;
    if (variant == RD_TREE_DIRECT && !direct_applies(s->p, s->progs.stack_depth)) return RD_ERR_UNSUPPORTED;
    s->tree_variant = int(variant);
    return RD_OK;
}

int rd_schedule_trace(const rd_schedule_t *s, uint64_t *t_ns, size_t cap_events)
{
    if (!s || !t_ns) return RD_ERR_INVALID_ARG;
    const size_t n = s->sched.events.size();
    if (cap_events < n) return RD_ERR_TOO_SMALL;
    if (!s->dev.f_traced) return RD_ERR_UNSUPPORTED;
    if (n > 0 && cudaMemcpy(t_ns, s->dev.f_trace, 3 * n * sizeof(uint64_t), cudaMemcpyDeviceToHost) != cudaSuccess) return RD_ERR_CUDA;
    return RD_OK;
}

int rd_schedule_faithful_shape(rd_schedule_t *s, int *blocks_per_process, int *slots_per_process, size_t *scratch_bytes)
{
    if (!s) return RD_ERR_INVALID_ARG;
    if (s->p < 2) {
        if (blocks_per_process) *blocks_per_process = 0;
        if (slots_per_process) *slots_per_process = 0;
        if (scratch_bytes) *scratch_bytes = 0;
        return RD_OK;
    }
    return guarded([&] {
        if (int rc = upload(s)) return rc;
        if (int rc = prepare_faithful(s)) return rc;
        if (blocks_per_process) *blocks_per_process = s->dev.f_lanes;
        if (slots_per_process) *slots_per_process = s->dev.f_slots;
        if (scratch_bytes) *scratch_bytes = size_t(s->p) * size_t(s->dev.f_slots) * size_t(s->dev.f_slot_elems) * 4;
        return int(RD_OK);
    });
}

int rd_schedule_tree_shape(rd_schedule_t *s, int *variant, int *blocks_per_sm, int *ring_stages, size_t *n_tiles)
{
    if (!s) return RD_ERR_INVALID_ARG;
    return guarded([&] {
        if (int rc = upload(s)) return rc;
        TreeLaunch l{};
        const int opsPerStage = stage_ops(1, s->tree_variant, s->progs.shared_depth);
        if (int rc = tiles_for(s, tiles_key(opsPerStage), &l.tiles, &l.n_tiles)) return rc;
        const bool direct = direct_applies(s->p, s->progs.stack_depth) &&
                            (s->tree_variant == RD_TREE_DIRECT || (s->tree_variant == RD_TREE_AUTO && s->p <= kDirectAutoProcs));
        if (variant) *variant = direct ? RD_TREE_DIRECT : opsPerStage == 2 ? RD_TREE_STREAM_PAIRED : RD_TREE_STREAM;
        const DeviceTables::StreamPlan *plan = nullptr;
        if (int rc = stream_plan(s, 1, opsPerStage, stage_warps(1, opsPerStage, s->progs.shared_depth, s->p), &plan)) return rc;
        if (blocks_per_sm) *blocks_per_sm = direct ? direct_blocks_per_sm(s->p) : plan->ctas_per_sm;
        if (ring_stages) *ring_stages = direct ? 0 : plan->stages;
        if (n_tiles) *n_tiles = l.n_tiles;
        return int(RD_OK);
    });
}

int rd_schedule_status(rd_schedule_t *s, int *device_status)
{
    if (!s || !device_status) return RD_ERR_INVALID_ARG;
    if (s->dev.device < 0) { *device_status = 0; return RD_OK; }     // nothing has run on a device yet
    int prev = -1, st = 0;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(s->dev.device) != cudaSuccess) return RD_ERR_CUDA;
    bool ok = cudaDeviceSynchronize() == cudaSuccess;
    ok = ok && cudaMemcpy(&st, s->dev.status, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess;
    if (ok && st != 0) {
        ok = cudaMemset(s->dev.status, 0, sizeof(int)) == cudaSuccess;
        reset_tile_counters(s->dev.device);          // the device is idle here
    }
    cudaSetDevice(prev);
    if (!ok) return RD_ERR_CUDA;
    *device_status = st;
    return RD_OK;
}

int rd_schedule_actions(const rd_schedule_t *s, int process, int32_t *buf, size_t cap_actions, size_t *n_actions, int *slots_per_process)
{
    if (!s || process < 0 || process >= s->p || (!buf && cap_actions > 0)) return RD_ERR_INVALID_ARG;
    ActionLists lists;
    try {
        if (int rc = build_actions(s->p, s->sched.seg_off.size() - 1, s->sched.events, lists)) return rc;
    } catch (const std::bad_alloc &) {
        return RD_ERR_NOMEM;
    }
    const uint32_t k0 = lists.first[size_t(process)], k1 = lists.first[size_t(process) + 1];
    if (n_actions) *n_actions = k1 - k0;
    if (slots_per_process) *slots_per_process = lists.slots_per_proc;
    if (cap_actions < k1 - k0) return RD_ERR_TOO_SMALL;
    for (uint32_t k = k0; k < k1; k++) {
        const Action &a = lists.actions[k];
        const int32_t v[8] = {a.seg, a.peer, a.kind, a.slot, a.peer_slot, a.first, a.event, a.wait_event};
        std::memcpy(buf + size_t(k - k0) * 8, v, sizeof(v));
    }
    return RD_OK;
}

int rd_reduce_faithful_static(rd_schedule_t *s, const void *const *d_inputs, void *d_out, size_t n_elems, rd_dtype_t dtype,
                              rd_op_t op, void *cuda_stream, rd_stats_t *stats)
{
    size_t n_words = 0;
    if (int rc = check_reduce_args(s, d_inputs, d_out, n_elems, dtype, op, &n_words)) return rc;
    if (is_half(dtype)) return RD_ERR_UNSUPPORTED;
    rd_stats_t st;
    std::memset(&st, 0, sizeof(st));
    st.bytes_moved = uint64_t(s->p + 1) * uint64_t(n_words) * 4u;
    st.predicted_s = double(s->sched.completion) * s->ticks.tick;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (n_elems == 0) { if (stats) *stats = st; return RD_OK; }
    if (s->p == 1) {
        if (d_out != d_inputs[0] && cudaMemcpyAsync(d_out, d_inputs[0], n_words * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
            return RD_ERR_CUDA;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return RD_ERR_CUDA;
        if (stats) *stats = st;
        return RD_OK;
    }
    return guarded([&]() -> int {
        ActionLists lists;
        const size_t q = s->sched.seg_off.size() - 1;
        if (int rc = build_actions(s->p, q, s->sched.events, lists)) return rc;
        std::vector<FaithfulAction> acts(lists.actions.size());
        for (size_t k = 0; k < acts.size(); k++) {
            const Action &a = lists.actions[k];
            acts[k] = FaithfulAction{a.seg, a.peer, a.kind, a.slot, a.peer_slot, a.first, a.event, a.wait_event};
        }
        std::vector<unsigned long long> times(2 * size_t(s->p) * 16);
        bool wide = (reinterpret_cast<uintptr_t>(d_out) & 15u) == 0;
        for (int i = 0; i < s->p && wide; i++) wide = (reinterpret_cast<uintptr_t>(d_inputs[i]) & 15u) == 0;
        StaticRun r{};
        r.p = s->p;
        r.h_actions = acts.data(); r.n_actions = acts.size();
        r.h_first = lists.first.data();
        r.h_seg_off = s->sched.seg_off.data(); r.n_seg_off = s->sched.seg_off.size();
        r.h_inputs = d_inputs; r.d_out = d_out;
        r.n_events = s->sched.events.size();
        r.slots = std::max(lists.slots_per_proc, 1);
        r.slot_elems = faithful_slot_words(s->sched.seg_off);
        r.blocking_send = s->port == RD_PORT_UNI ? 1 : 0;
        r.dtype = int(dtype); r.op = int(op); r.wide = wide;
        r.wait_seconds = s->wait_budget_s;
        r.stream = cuda_stream;
        r.h_block_times = times.data();
        const int rc = faithful_static_run(r);
        if (rc == 2) return RD_ERR_TOO_LARGE;
        if (rc == 3) return RD_ERR_UNSUPPORTED;
        if (rc != 0) return RD_ERR_CUDA;
        st.device_status = r.device_status;
        st.makespan_ns = r.makespan_ns;
        st.kernel_ms = r.makespan_ns * 1e-6;
        st.gbytes_per_s = r.makespan_ns > 0 ? double(st.bytes_moved) / r.makespan_ns : 0.0;
        st.n_launches = 1;
        if (stats) *stats = st;
        return r.device_status != 0 ? RD_ERR_TIMEOUT : RD_OK;
    });
}

int rd_search_segmentation(int p, size_t msg_bytes, size_t unit_bytes, const rd_model_t *model, size_t *seg_bytes, size_t cap,
                           size_t *q_out, int64_t *predicted_ticks)
{
    if (!model || !q_out || (!seg_bytes && cap > 0) || p < 1 || p > kMaxProcs) return RD_ERR_INVALID_ARG;
    Ticks t;
    if (int rc = make_ticks(model, t)) return rc;
    try {
        std::vector<int64_t> best;
        int64_t ticks = 0;
        if (int rc = search_segmentation(p, msg_bytes, unit_bytes, t, best, &ticks)) return rc;
        *q_out = best.size();
        if (predicted_ticks) *predicted_ticks = ticks;
        if (cap < best.size()) return RD_ERR_TOO_SMALL;
        for (size_t j = 0; j < best.size(); j++) seg_bytes[j] = size_t(best[j]);
    } catch (const std::bad_alloc &) {
        return RD_ERR_NOMEM;
    }
    return RD_OK;
}

void rd_destroy(rd_schedule_t *s)
{
    if (!s) return;
    release_device(s->dev);
    delete s;
}

const char *rd_strerror(int status)
{
    switch (status) {
    case RD_OK: return "success";
    case RD_ERR_INVALID_ARG: return "invalid argument";
    case RD_ERR_UNSUPPORTED: return "combination not supported";
    case RD_ERR_NOMEM: return "out of memory";
    case RD_ERR_CUDA: return "CUDA runtime call failed";
    case RD_ERR_TIMEOUT: return "a bounded wait inside a kernel gave up";
    case RD_ERR_SIZE_MISMATCH: return "n_elems does not match the schedule's message size";
    case RD_ERR_INTERNAL: return "generated schedule failed the consistency check";
    case RD_ERR_TOO_SMALL: return "output array too small";
    case RD_ERR_TOO_LARGE: return "the schedule needs more scratch than the built-in device array holds";
    }
    return "unknown status";
}

}  // extern "C"
