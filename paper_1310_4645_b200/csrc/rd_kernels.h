// Launch interface between the C ABI (host C++) and the CUDA kernels.
#ifndef RD_KERNELS_H_
#define RD_KERNELS_H_

#include <cstddef>
#include <cstdint>

namespace rd {

// One unit of work of the tree kernel: a run of elements inside one segment.
struct TileDesc {
    uint64_t elem_off;   // first element
    uint32_t len;        // elements in the tile (<= tile capacity)
    uint32_t prog;       // first word of the segment's program in the operation table
};

constexpr int kTreeThreads = 256;
constexpr int kPackedPtrs = 256;      // up to this many input pointers travel as kernel parameters

struct TreeLaunch {
    const void *const *host_ptrs;     // p device pointers (host array)
    const void *const *dev_ptr_table; // device copy of the same, used when p > kPackedPtrs
    void *out;
    const TileDesc *tiles;            // device
    const uint32_t *ops;              // device
    uint32_t n_tiles;
    int p;
    int stack_depth;                  // partial results a program keeps besides the running one
    int shared_depth;                 // levels the streaming kernel's shared-memory stack needs in this launch
    int dtype, op;                    // rd_dtype_t, rd_op_t
    int vec;                          // 4: 128-bit path, 1: element path
    int sm_count;
    int device;
    void *stream;
    // streaming variant only
    const uint32_t *cta_first;        // device: n_ctas + 1 offsets into tiles
    uint32_t n_ctas;
    int stages;
    int stage_elems;
    int ops_per_stage;                // operand tiles that share a ring stage (1 or 2); tiles hold stage_elems / ops_per_stage words
    int consumer_warps;               // 8, 4 or 2 (two tiles per stage: 4 or 2)
    int *status;                      // device word
    uint32_t *tile_counter;           // device: two words, both 0, for handing tiles out on demand; null: fixed ranges
};

// One reduction of a batch that runs as a single launch of the streaming kernel.
struct BatchJob {
    const uint32_t *const *inputs;    // device table of the job's p input pointers (batches that do not fit the parameters)
    uint32_t *out;
    const TileDesc *tiles;            // the tiles of the job's schedule (streaming path)
    const uint32_t *ops;              // its operation table
    uint32_t tile_begin, tile_end;    // the job's tiles are [tile_begin, tile_end) of the launch's tiles
    int p;
    int ptr_base;                     // first of the job's p pointers in the launch's pointer array (small batches)
};
constexpr int kBatchPackJobs = 16;    // a batch of at most this many jobs and kBatchPackPtrs input pointers
constexpr int kBatchPackPtrs = 1024;  // travels inside the kernel's parameters

struct BatchLaunch {
    const BatchJob *host_jobs;        // host: small batch, descriptors and pointers go into the parameters ...
    const void *const *host_ptrs;     //       ... n_ptrs device pointers, job after job
    uint32_t n_ptrs;
    const BatchJob *jobs;             // device, n_jobs entries (when host_jobs is null)
    uint32_t n_jobs, n_tiles;
    uint32_t n_ctas;
    int stages, stack_depth, stage_elems, ops_per_stage, consumer_warps;   // stack_depth: levels in shared memory
    int dtype, op, device;
    int *status;                      // device word
    uint32_t *tile_counter;           // as in TreeLaunch
    void *stream;
};
int launch_tree_stream_batch(const BatchLaunch &b);

// Elements one tile of the element-path kernel may hold for the given vector width.
uint32_t tree_tile_elems(int vec);
// Launches the tree kernel; returns a cudaError_t value (0 = success).
int launch_tree(const TreeLaunch &a);
// Streaming variant (128-bit path): stage size for a CTA's share of the message, ring shape for a
// stack depth and the SM's shared memory, launch.
int stream_stage_elems(uint64_t elems_per_cta);
// many_pushes: the programs push a partial result on the shared-memory stack for at least every tenth operand.
void stream_shape(int stack_depth, int acc_words, int ops_per_stage, bool many_pushes, int smem_per_sm, int stage_elems, uint64_t n_tiles,
                  int sm_count, int *ctas_per_sm, int *stages);
// Whether the streaming kernel of this shape runs the marked sub-expressions of a program in a second accumulator
// (its shared-memory stack then needs Programs::shared_depth levels, else Programs::stack_depth).
bool stream_second_accumulator(int acc_words, int ops_per_stage);
size_t stream_smem_bytes(int stages, int depth, int stage_elems, int acc_words, int ops_per_stage);
int launch_tree_stream(const TreeLaunch &a);
// Direct variant (128-bit path, at most kDirectMaxProcs processes): all operands of a thread's elements
// are fetched into registers at once.  Uses the streaming variant's tiles.
constexpr int kDirectMaxProcs = 8;
bool direct_applies(int p, int stack_depth);
int direct_blocks_per_sm(int p);
int launch_tree_direct(const TreeLaunch &a);

// Broadcast (all-reduce = reduce + broadcast; rd_broadcast.cu): copies n_words 32-bit words from src to each of the
// n_dst destinations (device pointers in a host array).  aligned: all buffers 16-byte aligned; the whole 128-bit
// vectors then go through bulk asynchronous copies, the last n_words mod 4 words (or, unaligned, everything) through a
// word-wise kernel.  status: device word that receives an error code when a bounded wait gives up.
// broadcast_launches: how many kernels launch_broadcast launches for these arguments.
constexpr int kBcastPackPtrs = 256;   // destinations per launch (they travel as kernel parameters)
int launch_broadcast(const void *src, void *const *dsts, int n_dst, uint64_t n_words, bool aligned, int sm_count, int *status,
                     void *stream);
int broadcast_launches(int n_dst, uint64_t n_words, bool aligned);

// ---- schedule-faithful execution (rd_faithful.cu)
constexpr int kFaithfulThreads = 128;

struct FaithfulAction {            // device copy of one step of a process (see rd::Action)
    int32_t seg, peer, kind, slot, peer_slot, first, event, wait_event;
};

struct FaithfulParams {
    const uint32_t *const *inputs;   // device table of the p input pointers
    uint32_t *out;
    uint32_t *scratch;               // [p][slots][slot_elems]
    const FaithfulAction *actions;   // all processes back to back
    const uint32_t *first;           // p+1 offsets into actions
    const uint64_t *seg_off;         // q+1 segment boundaries, elements
    uint32_t *posted, *taken;        // [n_events][lanes], hold the epoch of the launch that raised them
    unsigned long long *trace;       // [n_events][3]: receiver ready, transfer start, combine end (ns), lane 0 only
    unsigned long long *block_times; // [blocks][2]: first action start, last action end (ns)
    int *status;                     // 0 or RD_ERR_TIMEOUT
    int *abort_flag;
    long long wait_cycles;           // budget of one wait, SM clock cycles
    uint32_t epoch;
    int n_procs, lanes, slots;
    uint64_t slot_elems;
    int blocking_send;               // 1: a send waits until it has been taken (one port per process)
};

// Resident blocks per SM of the kernel variant (0 = success), and the cooperative launch itself.
int faithful_blocks_per_sm(int dtype, int op, bool wide, int *blocks_per_sm);
int launch_faithful(const FaithfulParams &prm, int dtype, int op, bool wide, void *stream);

// ---- the same kernel run entirely out of a fixed device array (no device allocation)
struct StaticRun {
    // in
    int p;
    const FaithfulAction *h_actions; size_t n_actions;   // host
    const uint32_t *h_first;                              // host, p + 1
    const uint64_t *h_seg_off; size_t n_seg_off;          // host
    const void *const *h_inputs;                          // host array of p device pointers
    void *d_out;
    size_t n_events;
    int slots; uint64_t slot_elems;
    int blocking_send, dtype, op;
    bool wide;
    double wait_seconds;
    void *stream;
    unsigned long long *h_block_times;                    // host scratch, 2 * p * 16 values
    // out
    size_t needed_bytes;
    int device_status, lanes;
    double makespan_ns;
};
size_t faithful_static_capacity();
// 0 done, 1 a CUDA call failed, 2 the schedule needs more than the array holds, 3 too many processes to be resident
int faithful_static_run(StaticRun &r);

}  // namespace rd
#endif
