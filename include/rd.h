/*
 * rd.h -- C ABI of the schedule-exact pipelined reduction library (librd.so).
 *
 * The library reduces the messages of p "processes" (p buffers of n 4- or
 * 8-byte elements in the memory of ONE GPU) into a root buffer, combining entry-wise
 * in exactly the order a reduction schedule fixes.  Schedules follow
 * Lowery & Langou, "A Greedy Algorithm for Optimally Pipelining a Reduction":
 * uni-greedy (Algorithm 1), bi-greedy (Algorithm 2), and the algorithms the
 * paper compares them with: binomial, pipeline, binary tree (Section IV) and
 * the reduce-scatter/gather butterfly (Section III).
 *
 * Conventions
 *   - Every function returns RD_OK (0) or a negative rd_status_t; nothing
 *     aborts, nothing throws across this boundary, and output arguments are
 *     left untouched on failure.
 *   - Processes are numbered 0..p-1 and the root is process 0 (the paper's
 *     implementation makes the same restriction, Fig. 2 caption).  The system
 *     is homogeneous and fully connected (Section II), so a schedule does not
 *     care which buffer plays which process: to reduce towards another root,
 *     pass the pointer array permuted so that the root's buffer comes first
 *     (the combine order is then the schedule's with the processes relabelled
 *     the same way).  rd_allreduce gives every process a copy of the result.
 *   - Sizes called "bytes" are bytes.  A schedule knows sizes in bytes only and reports segment
 *     boundaries in 4-byte words; n_elems of the reducing calls counts elements of the call's
 *     rd_dtype_t (4 or 8 bytes each).
 *   - "host" / "device" in a comment says where a pointer must point.
 *   - Times of the linear model (Section II): a message of b bytes costs
 *     alpha + beta*b, combining it costs gamma*b.  Internally time is an exact
 *     integer count of `tick` seconds, so that equal times are decided the
 *     same way everywhere: t_comm = round(alpha/tick) + round(beta/tick)*b,
 *     t_comp = round(gamma/tick)*b.
 *   - A communication must take time: a model whose alpha and beta both round to zero ticks is
 *     refused with RD_ERR_INVALID_ARG (every send would start and end at time 0 and the order of the
 *     events, hence of the combines, would be undefined).  gamma may be zero.
 *   - Thread safety: distinct schedules may be used from distinct threads.
 *     One schedule may be used by one thread at a time.
 */
#ifndef RD_H_
#define RD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define RD_API __attribute__((visibility("default")))
#else
#define RD_API
#endif

typedef struct rd_schedule rd_schedule_t; /* opaque; owns its host and device tables */

typedef enum {
    RD_OK = 0,
    RD_ERR_INVALID_ARG = -1,   /* null pointer, p < 1, size not a multiple of 4, unknown enum, ...      */
    RD_ERR_UNSUPPORTED = -2,   /* a combination the method does not define (see rd_schedule_create)     */
    RD_ERR_NOMEM = -3,         /* host or device allocation failed                                      */
    RD_ERR_CUDA = -4,          /* a CUDA runtime call failed (including: no device, no driver)          */
    RD_ERR_TIMEOUT = -5,       /* a bounded wait inside a kernel (tree mode or schedule-faithful) gave up */
    RD_ERR_SIZE_MISMATCH = -6, /* n_elems * element size differs from the schedule's message size       */
    RD_ERR_INTERNAL = -7,      /* a generated schedule failed the library's own consistency check       */
    RD_ERR_TOO_SMALL = -8,     /* an output array passed by the caller is too short                     */
    RD_ERR_TOO_LARGE = -9      /* rd_reduce_faithful_static: more scratch needed than its fixed array has */
} rd_status_t;

typedef enum {
    RD_UNI_GREEDY = 0, /* Algorithm 1; unidirectional ports only                                 */
    RD_BI_GREEDY = 1,  /* Algorithm 2; bidirectional ports only                                  */
    RD_BINOMIAL = 2,   /* Section IV; either port model                                          */
    RD_PIPELINE = 3,   /* Section IV; either port model                                          */
    RD_BINARY = 4,     /* Section IV; either port model                                          */
    RD_BUTTERFLY = 5   /* Section III (reduce-scatter/gather); bidirectional ports only           */
} rd_algo_t;

typedef enum { RD_PORT_UNI = 0, RD_PORT_BI = 1 } rd_port_t;   /* Section II */
/* Entry-wise operation (associative and commutative, as the method requires).  Integer sum and product
 * wrap modulo 2^32 (2^64 for RD_INT64); max / min keep the held value on ties (incoming > held ? incoming : held), which
 * settles the sign of a zero result; fp32 and fp64 sum and product are one IEEE
 * round-to-nearest operation per combine (subnormals kept, infinities as IEEE has them).  A NaN, whether an
 * input or born of inf - inf or inf * 0, comes out as a NaN of the GPU's own bit pattern (0x7fffffff), which
 * need not be the pattern another machine produces; under max and min every comparison with a NaN is false,
 * so an incoming NaN never replaces the held value and a held NaN is never replaced. */
typedef enum { RD_SUM = 0, RD_MAX = 1, RD_MIN = 2, RD_PROD = 3 } rd_op_t;
/* Element type.  The paper's implementation is restricted to int and notes that the restriction is
 * not a consequence of the algorithm (Fig. 2 caption).  With an 8-byte type no segment may begin
 * inside an element: msg_bytes and every segment size multiples of 8 (for the butterfly, whose
 * chunks come from halving the message: n_elems a multiple of the largest power of two <= p);
 * rd_optimal_segment returns multiples of 4, round them up.  Otherwise the reducing calls return
 * RD_ERR_INVALID_ARG.
 *
 * RD_BF16, RD_FP16: bf16 / IEEE binary16 elements combined in fp32 (the usual "16-bit storage, 32-bit
 * accumulation"; the paper fixes nothing here).  Every input is widened exactly, partial results are fp32
 * values combined by one IEEE fp32 operation per combine in the schedule's order, and only what the root
 * holds at the end is rounded to 16 bits, once, to nearest with ties to even (fp16: overflow to infinity,
 * gradual underflow).  (Max and min select one of their operands, so the kernels take them on the 16-bit values
 * directly; the bits are the same.)  n_elems counts 16-bit elements (msg_bytes / 2, always even); buffers must be aligned
 * to 4 bytes.  Tree mode only: the schedule-faithful execution would have to hand fp32 partial segments
 * between processes and returns RD_ERR_UNSUPPORTED. */
typedef enum { RD_INT32 = 0, RD_FP32 = 1, RD_INT64 = 2, RD_FP64 = 3, RD_BF16 = 4, RD_FP16 = 5 } rd_dtype_t;
typedef enum { RD_EXEC_TREE = 0, RD_EXEC_FAITHFUL = 1 } rd_exec_t;

/* Linear model of Section II.  alpha in seconds, beta and gamma in seconds per
 * byte, tick = seconds per integer time unit (0 selects 1e-15).  alpha/tick,
 * beta/tick and gamma/tick are rounded to the nearest integer.               */
typedef struct { double alpha, beta, gamma, tick; } rd_model_t;

/* One send/receive pair (Section V: reduce(X, S, a, b, t)): process src sends
 * segment seg to process dst starting at tick t_start.  kind 0: dst combines
 * what it holds (left operand) with what arrives; kind 1: dst only stores it
 * (gather phase of the butterfly).  For the butterfly a "segment" is the final
 * chunk of the message that one process owns after the reduce-scatter.        */
typedef struct { int32_t seg, src, dst, kind; int64_t t_start; } rd_event_t;

/* Filled by rd_reduce when requested.  Asking for it makes the call wait for
 * the kernel.                                                                 */
typedef struct {
    double kernel_ms;      /* device time of the kernel(s), CUDA events                       */
    double gbytes_per_s;   /* (p*m + m) bytes / kernel time, in 1e9 bytes per second          */
    double makespan_ns;    /* faithful mode: first action start to the root's last combine    */
    double predicted_s;    /* the schedule's completion time under the linear model           */
    uint64_t bytes_moved;  /* p*m + m                                                         */
    int32_t device_status; /* faithful mode: 0, or RD_ERR_TIMEOUT                             */
    int32_t n_launches;    /* kernels launched by this call                                   */
} rd_stats_t;

/*
 * rd_schedule_create -- Sections II, IV, V (Algorithm 1), VI (Algorithm 2), III.
 * Generates the schedule for p processes and a message of msg_bytes per
 * process, cut into equal segments of seg_bytes with a possibly smaller last
 * one (Section II), and compiles it into per-segment combine programs.  Host
 * work only: no CUDA call is made, so it works without a GPU.
 *   out        host; receives the new schedule; release with rd_destroy.
 *   algo/port  legal pairs: uni-greedy + UNI; bi-greedy + BI; butterfly + BI;
 *              binomial, pipeline, binary + either.  Others: RD_ERR_UNSUPPORTED.
 *   p          1..4096.  Butterfly: when p is not a power of two the processes beyond
 *              the largest power of two P first send their whole message to a
 *              partner below P (one extra round), then the butterfly runs on P
 *              processes; the schedule then has P chunks ("segments").
 *   msg_bytes  multiple of 4; may be 0.
 *   seg_bytes  multiple of 4, 0 < seg_bytes; values above msg_bytes mean one
 *              segment.  0 selects the segment size rd_optimal_segment gives.
 *              Ignored by the butterfly, which halves the message instead.
 *              Binomial: the paper uses one segment (seg_bytes = 0 gives
 *              that); several segments are reduced one after the other, each
 *              by the same tree.
 *   model      host; must not be NULL.
 */
RD_API int rd_schedule_create(rd_schedule_t **out, rd_algo_t algo, rd_port_t port, int p,
                       size_t msg_bytes, size_t seg_bytes, const rd_model_t *model);

/*
 * rd_schedule_create_segments -- Section VIII (unequal segmentation).
 * As rd_schedule_create, with the q segment sizes given one by one (each a
 * positive multiple of 4 bytes; their sum is the message size).  Algorithm 1
 * is defined for any segmentation; the lock-step algorithms use the largest
 * segment as their round length.  Not available for the butterfly.
 *   seg_bytes  host array of q sizes.
 */
RD_API int rd_schedule_create_segments(rd_schedule_t **out, rd_algo_t algo, rd_port_t port, int p,
                                const size_t *seg_bytes, size_t q, const rd_model_t *model);

/*
 * rd_optimal_segment -- Table I and Table III (s_opt rows), Section VII.
 * The equal segment size, in bytes (multiple of 4, 4 <= s <= msg_bytes), that
 * minimises the schedule's completion time under `model`: the closed forms of
 * the tables for pipeline, binary and bi-greedy (the better of the two
 * integer segment counts around the real optimum; the whole message when the
 * formula's denominator is not positive), the whole message for binomial, a
 * search over powers of two for uni-greedy (the paper's tuning protocol), and
 * the whole message for the butterfly (it ignores the value).
 */
RD_API int rd_optimal_segment(rd_algo_t algo, rd_port_t port, int p, size_t msg_bytes,
                       const rd_model_t *model, size_t *seg_bytes_out);

/* rd_schedule_info -- Section V: the completion time is the final state of the
 * root.  Any output pointer may be NULL.  q is the number of segments (for the
 * butterfly: p chunks), n_events the number of send/receive pairs
 * ((p-1)*q for the tree schedules), predicted_ticks / predicted_seconds the
 * completion time under the model, stack_depth the number of partial results
 * the combine programs keep besides the running one on a plain stack (with the
 * hints of rd_schedule_program a kernel needs one level less).               */
RD_API int rd_schedule_info(const rd_schedule_t *s, int *p, size_t *q, size_t *n_events,
                     double *predicted_seconds, int64_t *predicted_ticks, int *stack_depth);

/* rd_schedule_events -- copies the n_events pairs into buf (host, capacity cap
 * entries) ordered by (t_start, seg, src, dst).  RD_ERR_TOO_SMALL if cap is
 * too small.                                                                  */
RD_API int rd_schedule_events(const rd_schedule_t *s, rd_event_t *buf, size_t cap);

/* rd_schedule_segments -- writes the q+1 segment boundaries in elements into
 * off (host, capacity cap entries): segment j is elements [off[j], off[j+1]). */
RD_API int rd_schedule_segments(const rd_schedule_t *s, uint64_t *off, size_t cap);

/*
 * rd_schedule_program -- the compiled combine program of one segment (what the
 * tree kernel interprets), for inspection and for checking it on the host.
 * Writes its p operations to ops (host, capacity cap) and returns RD_OK, or
 * RD_ERR_TOO_SMALL.  An operation is a 32-bit word:
 *   bits  0-11  process whose element is loaded
 *   bits 12-13  0 LOAD      top = x
 *               1 PUSH_LOAD push top; top = x
 *               2 ACC_IN    top = combine(held = top, incoming = x)
 *               3 ACC_HELD  top = combine(held = x,   incoming = top)
 *   bits 14-17  npop: number of pops that follow
 *   bits 18-29  bit k = role of the k-th pop: 1: top = combine(held = popped, incoming = top)
 *                                              0: top = combine(held = top, incoming = popped)
 *   bit  30     the operation belongs to a sub-expression that needs no stack: it begins with a PUSH_LOAD,
 *               continues with ACC operations and ends with the operation that has bit 31 set, whose
 *               first pop takes back the entry the PUSH_LOAD pushed; nothing else is pushed or popped in
 *               between.  An interpreter may evaluate such a sub-expression in a second accumulator
 *               (PUSH_LOAD: second = x; ACC: second = combine(second, x) resp. combine(x, second)) and
 *               leave top where it is; at the end the pop's two values are top (as "popped") and second.
 *   bit  31     last operation of such a sub-expression
 * Bits 30 and 31 are hints: an interpreter that pushes and pops everything on one stack gets the same
 * result.  combine(held, incoming) = held + incoming, held * incoming, or incoming > held ? incoming : held
 * (min: <).
 * After the last operation top is the root's value (Section IV: the receiver
 * combines its segment with the one received).
 */
RD_API int rd_schedule_program(const rd_schedule_t *s, size_t seg, uint32_t *ops, size_t cap);

/*
 * rd_reduce -- the reduction itself (Section III "Reduce"; Section IV).
 *   d_inputs  HOST array of p DEVICE pointers; d_inputs[i] is process i's
 *             message of n_elems elements.  Never written.
 *   d_out     DEVICE; n_elems elements; receives what the root holds at the
 *             end.  May alias d_inputs[0] in tree mode only.
 *   n_elems   must equal the schedule's msg_bytes / element size (RD_ERR_SIZE_MISMATCH).
 *   exec      RD_EXEC_TREE: one kernel evaluates, per element, the segment's
 *             combine program in registers; asynchronous on cuda_stream.
 *             RD_EXEC_FAITHFUL: a persistent kernel in which groups of thread
 *             blocks play the processes and hand partial segments to each
 *             other through device memory, action by action; the call waits
 *             for it and reports its makespan.  Needs scratch memory, which
 *             the schedule allocates on first use and keeps.
 *   cuda_stream  a cudaStream_t (NULL = the legacy default stream).
 *   stats     host, or NULL.
 * The first call on a schedule uploads its tables to the current device
 * (allocates device memory, synchronises); rd_schedule_upload does the same
 * ahead of time.  The first tree-mode call on a device also allocates 512 KiB of counters there,
 * kept until the process ends: a launch of the streaming kernel hands its tiles to its thread
 * blocks on demand through one of them (a launch recorded into a CUDA graph uses none and gives
 * every thread block a fixed range of tiles instead).  After one such call per schedule, element type and operation, a
 * tree-mode call with at most 256 processes is a single kernel launch and may be
 * recorded into a CUDA graph (so may an rd_reduce_batch call of at most 16 aligned jobs with at most
 * 1024 input pointers in all, after one ordinary call of it).  Buffers must be aligned to the element; 16-byte aligned buffers take
 * the 128-bit streaming path (segments may start and end anywhere; when the message is
 * not a multiple of 16 bytes the last elements are done by a second, tiny launch), other
 * buffers a slower element-wise path.
 */
RD_API int rd_reduce(rd_schedule_t *s, const void *const *d_inputs, void *d_out, size_t n_elems,
              rd_dtype_t dtype, rd_op_t op, rd_exec_t exec, void *cuda_stream, rd_stats_t *stats);

/*
 * rd_allreduce -- Section III "All-reduce": every process ends up with the combined vector; as the paper
 * states it, a reduce followed by a broadcast.  Tree mode: the reduction of rd_reduce into d_outs[0] (the
 * root's copy, same kernel, same bits), then a broadcast kernel that copies the root's result to the other
 * p - 1 buffers.  When every copy is 16-byte aligned: for up to 16 destinations tiles of 4 KB travel through
 * shared memory by bulk asynchronous copies (one in, p - 1 out), for more every thread carries 128-bit vectors
 * through registers; the last n mod 4 words of a ragged message go by a second, word-wise launch.  Otherwise
 * word by word.  At most 256 destinations per launch.  Asynchronous on cuda_stream; a bounded wait that gives
 * up is reported as for rd_reduce (rd_schedule_status).
 *   d_inputs  HOST array of p DEVICE pointers, as in rd_reduce.
 *   d_outs    HOST array of p DEVICE pointers: d_outs[i] receives process i's copy, n_elems elements.
 *             d_outs[i] may be d_inputs[i] itself (in-place all-reduce); otherwise no copy may overlap any
 *             input or another copy (RD_ERR_INVALID_ARG).
 *   stats     host or NULL: kernel_ms covers both kernels; bytes_moved = p*m + m for the reduce plus
 *             m read and (p-1)*m written by the broadcast.
 */
RD_API int rd_allreduce(rd_schedule_t *s, const void *const *d_inputs, void *const *d_outs, size_t n_elems,
                        rd_dtype_t dtype, rd_op_t op, void *cuda_stream, rd_stats_t *stats);

/*
 * rd_reduce_batch -- several independent tree-mode reductions issued together (the paper has no
 * counterpart; Section VII runs the same messages under every schedule, and a library user reduces
 * many buffers).  Job j reduces d_inputs[j][0..p_j) into d_outs[j] under schedules[j]; all jobs share
 * dtype, op and stream.  Results are exactly those of n_jobs rd_reduce calls, and the batch as a whole
 * is ordered after what precedes it on cuda_stream and before what follows it.
 *   When every buffer of every job is 16-byte aligned and every message a whole number of 128-bit
 *   vectors, the batch is ONE launch of the streaming kernel: the tiles of all jobs are dealt to the
 *   thread blocks as if they were one reduction, so the batch pays one launch, one ring fill and one
 *   tail instead of n_jobs (measured on B200, 16 jobs of p = 64 with 1 MiB messages: about twice the
 *   throughput of 16 calls; 32 jobs with 256 KiB messages: about five times).  A batch of at most 16
 *   jobs with at most 1024 input pointers in all carries its job descriptors and pointers inside the
 *   kernel's parameters and copies nothing ahead of the launch; a larger one sends them to the device in
 *   one small copy from a pinned ring that a device's first such batch allocates (it grows when a batch
 *   needs more).  A bounded wait that gives up is reported through rd_schedule_status of the first
 *   job's schedule.
 *   Otherwise the jobs are issued alternately on two streams of the library's own, so that one job's
 *   thread blocks take the SM slots another job frees while its last blocks are still running (event
 *   fork and join around them; streams and events are created on a device's first such batch and kept).
 *   schedules, d_inputs, d_outs, n_elems   HOST arrays of n_jobs entries (d_inputs[j]: HOST array of
 *             DEVICE pointers as in rd_reduce).  The same schedule may serve several jobs.
 * RD_ERR_INVALID_ARG when a job's output overlaps another job's output or inputs (a job's output may
 * alias its own root input); otherwise the errors of rd_reduce.  On an error jobs before the failing
 * one may have been launched.
 */
RD_API int rd_reduce_batch(size_t n_jobs, rd_schedule_t *const *schedules, const void *const *const *d_inputs,
                    void *const *d_outs, const size_t *n_elems, rd_dtype_t dtype, rd_op_t op, void *cuda_stream);

/* rd_schedule_upload -- copies the schedule's tables to the current device now. */
RD_API int rd_schedule_upload(rd_schedule_t *s);

/*
 * rd_reduce_host -- rd_reduce (tree mode) for messages that live in HOST memory.
 *   h_inputs  HOST array of p HOST pointers (pinned memory makes the copies
 *             asynchronous; messages that follow each other in memory, such as
 *             the rows of one array, travel in one copy); h_out HOST, n_elems elements.
 *   d_staging DEVICE; (p + 1) * n_elems elements of scratch owned by the
 *             caller: the p messages are copied there, reduced, and the
 *             result copied back.  The call returns after the result is in
 *             h_out.
 */
RD_API int rd_reduce_host(rd_schedule_t *s, const void *const *h_inputs, void *h_out, void *d_staging,
                   size_t n_elems, rd_dtype_t dtype, rd_op_t op, void *cuda_stream);

/*
 * rd_schedule_set_wait_budget -- the longest a block of the schedule-faithful kernel waits for
 * another process before it gives up (default 2 s, at most 60 s).  When a wait runs out the
 * kernel ends by itself, rd_reduce returns RD_ERR_TIMEOUT and the schedule stays usable.  The
 * paper has no counterpart: its processes block in MPI_Recv.
 */
RD_API int rd_schedule_set_wait_budget(rd_schedule_t *s, double seconds);

/*
 * rd_schedule_set_tree_variant -- which kernel serves tree-mode calls whose buffers are all 16-byte
 * aligned (the paper has no counterpart; the result is the same bit for bit).
 *   RD_TREE_AUTO    the library chooses (default; at present always the streaming kernel, which is
 *                   the faster one for every process count).
 *   RD_TREE_STREAM  operand tiles are streamed through a shared-memory ring by bulk asynchronous
 *                   copies; any number of processes.
 *   RD_TREE_DIRECT  every thread fetches all p operands of its elements into registers at once; at
 *                   most 8 processes (RD_ERR_UNSUPPORTED beyond); 4- and 8-byte element types.
 *   RD_TREE_STREAM_PAIRED  the streaming kernel on tiles of half the length (1024 words), a ring stage
 *                   holding the tiles of two consecutive operands: the partial results that wait in the
 *                   stack take half the shared memory per tile, the bytes per stage hand-over stay the same.
 *                   What RD_TREE_AUTO picks for sums and products of the 16-bit element types (whose partial
 *                   results are fp32) when the programs keep two or more partial results waiting.
 */
typedef enum { RD_TREE_AUTO = 0, RD_TREE_STREAM = 1, RD_TREE_DIRECT = 2, RD_TREE_STREAM_PAIRED = 3 } rd_tree_variant_t;
RD_API int rd_schedule_set_tree_variant(rd_schedule_t *s, rd_tree_variant_t variant);

/*
 * rd_schedule_tree_shape -- how a tree-mode call with 16-byte aligned buffers will run this schedule on
 * the current device with a 4- or 8-byte element type (the paper has no counterpart): the kernel
 * (RD_TREE_STREAM, RD_TREE_STREAM_PAIRED or RD_TREE_DIRECT), its thread blocks per SM, the stages of the
 * streaming kernel's shared-memory ring (0 for the direct kernel) and the number of tiles the message is cut
 * into (runs of at most 2048 4-byte words inside one segment; 1024 for RD_TREE_STREAM_PAIRED).
 * Uploads the schedule's tables if they are not on the device yet.  Any output pointer may be NULL.
 */
RD_API int rd_schedule_tree_shape(rd_schedule_t *s, int *variant, int *blocks_per_sm, int *ring_stages, size_t *n_tiles);

/*
 * rd_schedule_trace -- measured times of the last schedule-faithful rd_reduce, to set against
 * the model's alpha + beta*s (+ gamma*s) per pair (Section V).  For every send/receive pair, in
 * the order of rd_schedule_events, three values in nanoseconds of the GPU's global timer, taken by
 * the receiver's first block: when the receiver was ready for the pair, when the sender's data
 * became available to it, and when the combined segment was written.
 *   t_ns  host; 3 * n_events values; cap_events = capacity in pairs (RD_ERR_TOO_SMALL).
 * RD_ERR_UNSUPPORTED before any schedule-faithful run.
 */
RD_API int rd_schedule_trace(const rd_schedule_t *s, uint64_t *t_ns, size_t cap_events);

/*
 * rd_schedule_faithful_shape -- how the schedule-faithful kernel will run this schedule on the
 * current device: thread blocks per process, scratch slots per process (Section V: a process that
 * has received but not yet sent a segment must keep its partial result; uni-greedy needs one such
 * buffer, bi-greedy more, Section VI-B) and the bytes of scratch the schedule allocates for them.
 * Allocates that scratch if it has not been allocated yet.  Any output pointer may be NULL.
 */
RD_API int rd_schedule_faithful_shape(rd_schedule_t *s, int *blocks_per_process, int *slots_per_process,
                                      size_t *scratch_bytes);

/*
 * rd_schedule_actions -- what one process does in the schedule-faithful execution: its own sends
 * and receives in start-time order (Section IV: sending and receiving processors are paired; after
 * a processor sends a segment it is reduced for it).  Host work only.  Each action is 8 int32:
 *   seg, peer, kind (0 receive and combine, 1 receive and store, 2 send),
 *   slot (where this process keeps its value of the segment: >= 0 scratch slot, -1 its input,
 *   -2 the output buffer), peer_slot (receive: the same for the sender), first (receive: 1 when
 *   the held operand is this process's own input), event (index of the pair in
 *   rd_schedule_events), wait_event (receive into a recycled slot: the pair that must have been
 *   taken before the slot is overwritten, else -1).
 *   buf host, capacity cap_actions actions; n_actions / slots_per_process may be NULL.
 * RD_ERR_TOO_SMALL leaves buf untouched but still reports n_actions.
 * On the GPU a process is played by G thread blocks that never synchronise with each other.  A
 * segment that begins at 4-byte word b of the message sits in its scratch slot from word b mod 4 on,
 * so that slot and messages agree on where the 128-bit boundaries fall; a slot has W words, the
 * largest (b mod 4) + length over the segments, rounded up to a multiple of 4.  Block g works on slot
 * words [U*g/G, U*(g+1)/G) * v, clipped to the segment, with v = 4 words when all buffers are
 * 16-byte aligned (else one element) and U = W / v: the same slot words for every segment, so that
 * blocks which are at different points of the schedule never meet in a scratch slot.
 */
RD_API int rd_schedule_actions(const rd_schedule_t *s, int process, int32_t *buf, size_t cap_actions,
                               size_t *n_actions, int *slots_per_process);

/*
 * rd_reduce_faithful_static -- the schedule-faithful reduction for callers that must not allocate
 * device memory.  (The paper has no counterpart; this exists for the library's users.)
 *
 * Who needs it: code that runs after a framework has claimed all device memory for its own pool
 * (an inference server, a training job sized to the last byte) and would get cudaErrorMemoryAllocation
 * from any cudaMalloc; code in a latency-critical loop, where an allocation may take the driver's
 * global lock and stall every stream; code that is not allowed to change the process's memory
 * footprint at run time.  rd_reduce in RD_EXEC_FAITHFUL mode allocates its tables, flags and partial
 * result slots with cudaMalloc on first use; this entry point instead keeps all of that in one
 * device array of 32 MiB that is part of the library image (every GPU that loads librd.so holds
 * these 32 MiB until the process exits).  It calls no cudaMalloc / cudaFree and nothing that
 * allocates device memory; it does not touch the device tables rd_reduce keeps for the schedule.
 *
 * Arguments and result are those of rd_reduce(..., RD_EXEC_FAITHFUL, ...): same kernel, same bits.
 * stats (host, may be NULL): makespan_ns, predicted_s, bytes_moved, device_status, n_launches;
 * kernel_ms and gbytes_per_s are derived from the makespan.  The call returns when the result is
 * in d_out.
 *
 * Limits and rules
 *   - The schedule's tables (32 bytes per action, two actions per send/receive pair), 8 bytes of
 *     flags per pair and block, 24 bytes of time stamps per pair, and p x slots x largest-segment
 *     bytes of partial results must fit in the 32 MiB together: otherwise RD_ERR_TOO_LARGE and
 *     nothing is launched.  (Example: p = 64, 256 segments of 16 KiB, uni-greedy: about 5 MiB.)
 *   - The first call on a device looks up the array's device address (the device must be current);
 *     make that first call outside any stream capture.
 *   - All calls, of all schedules and threads, share the one array, and it still holds the previous
 *     call's contents: the entry point clears the flags, status words and time stamps itself at the
 *     start of every call, but two calls that overlap on the GPU (different streams or threads)
 *     corrupt each other.  Issue them one after the other.
 */
RD_API int rd_reduce_faithful_static(rd_schedule_t *s, const void *const *d_inputs, void *d_out, size_t n_elems,
                                     rd_dtype_t dtype, rd_op_t op, void *cuda_stream, rd_stats_t *stats);

/*
 * rd_search_segmentation -- Section VIII (unequal segmentation) for uni-greedy, which is optimal for
 * any given segmentation (Theorem 5) but whose best segmentation need not be an equal one.  Starts from
 * every best equi-segmentation in multiples of unit_bytes and moves one unit at a time between segments
 * (or splits one off), looking two moves ahead when no single move helps, while the completion time
 * under `model` gets shorter; the paper observes that the optimum usually lies one or two such moves
 * from the best equi-segmentation.  Host work only.
 *   msg_bytes  a multiple of unit_bytes; unit_bytes a multiple of 4; at most 4096 units.
 *   seg_bytes  host, capacity cap sizes; q_out receives the number of segments (also when cap is too
 *              small: RD_ERR_TOO_SMALL); predicted_ticks (may be NULL) the completion time.
 * Feed the result to rd_schedule_create_segments.
 */
RD_API int rd_search_segmentation(int p, size_t msg_bytes, size_t unit_bytes, const rd_model_t *model,
                                  size_t *seg_bytes, size_t cap, size_t *q_out, int64_t *predicted_ticks);

/*
 * rd_schedule_status -- tree-mode calls are asynchronous, so a kernel that had to give up a bounded
 * wait (see rd_schedule_set_wait_budget; it should never happen) cannot report it through rd_reduce's
 * return value.  This waits for the schedule's device to be idle and returns the status word its
 * kernels share: 0, or RD_ERR_TIMEOUT if some launch since the last query gave up (its output is then
 * not valid); the word is cleared.  The paper has no counterpart.
 */
RD_API int rd_schedule_status(rd_schedule_t *s, int *device_status);

/* rd_destroy -- frees the schedule and its device tables.  NULL is allowed. */
RD_API void rd_destroy(rd_schedule_t *s);

/* rd_strerror -- static, never NULL. */
RD_API const char *rd_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* RD_H_ */
