// Internal declarations shared by the library's translation units (host side).
#ifndef RD_INTERNAL_H_
#define RD_INTERNAL_H_

#include <cstddef>
#include <cstdint>
#include <vector>

#include "rd.h"

namespace rd {

// Linear model in integer ticks (Section II): t_comm(b) = A + B*b, t_comp(b) = G*b.
struct Ticks {
    int64_t A = 0, B = 0, G = 0;
    double tick = 1e-15;
    int64_t comm(int64_t bytes) const { return A + B * bytes; }
    int64_t comp(int64_t bytes) const { return G * bytes; }
};

struct Schedule {
    std::vector<rd_event_t> events;   // ordered by (t_start, seg, src, dst)
    std::vector<uint64_t> seg_off;    // q+1 boundaries, in elements
    int64_t completion = 0;           // ticks
};

// ---- rd_sched.cpp: Algorithm 1, Algorithm 2, Section IV trees, Section III butterfly
int gen_uni_greedy(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, Schedule &out, bool want_events);
int gen_bi_greedy(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, Schedule &out, bool want_events);
int gen_binomial(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, Schedule &out);
int gen_pipeline(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, bool bidir, Schedule &out);
int gen_binary(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, bool bidir, Schedule &out);
int gen_butterfly(int p, uint64_t n_elems, const Ticks &c, Schedule &out);
void sort_events(std::vector<rd_event_t> &ev);
int optimal_segment(rd_algo_t algo, rd_port_t port, int p, size_t msg_bytes, const Ticks &c, size_t *out);
int ceil_log2(uint64_t v);
int search_segmentation(int p, size_t msg_bytes, size_t unit, const Ticks &c, std::vector<int64_t> &best, int64_t *bestTicks);

// ---- rd_compile.cpp: events -> per-segment combine trees -> interpreter programs
constexpr int kIdxBits = 12;           // process index field of an operation word
constexpr int kMaxProcs = 1 << kIdxBits;
constexpr int kMaxPops = 12;
enum OpKind : uint32_t { OP_LOAD = 0, OP_PUSH_LOAD = 1, OP_ACC_IN = 2, OP_ACC_HELD = 3 };
constexpr uint32_t kOpSecondAccumulator = 1u << 30;   // the operation belongs to a sub-expression that needs no stack (see rd.h)
constexpr uint32_t kOpMergeSecond = 1u << 31;         // ... and is its last one: its first pop joins it with the running value

struct Programs {
    std::vector<uint32_t> ops;        // distinct programs, p words each, back to back
    std::vector<uint32_t> seg_prog;   // per segment: first word of its program in ops
    int stack_depth = 0;              // deepest stack any program needs (entries besides top)
    int shared_depth = 0;             // ... when sub-expressions that need no stack run in a second accumulator
    size_t shared_pushes = 0;         // pushes that remain then, summed over all segments
    size_t n_distinct = 0;
};
int compile_programs(int p, size_t q, const std::vector<rd_event_t> &events, Programs &out);

// One step of a process in the schedule-faithful execution.
struct Action {
    int32_t seg;         // segment (index into seg_off)
    int32_t peer;        // the other process
    int32_t kind;        // 0 receive and combine, 1 receive and store, 2 send
    int32_t slot;        // where this process keeps its value of the segment: >= 0 a scratch slot,
                         // -1 its own input (a send of a segment it never received), -2 the output (root)
    int32_t peer_slot;   // receive: where the sender keeps the value it sends (same encoding)
    int32_t first;       // receive: 1 when the held operand is the process's own input
    int32_t event;       // index of the send/receive pair in the schedule's event list (its flags)
    int32_t wait_event;  // receive into a recycled slot: the pair that must have been taken first, or -1
};
struct ActionLists {
    std::vector<Action> actions;      // all processes back to back, each in start-time order
    std::vector<uint32_t> first;      // p+1 offsets
    int slots_per_proc = 0;           // scratch slots (of one largest segment each) a process needs
};
int build_actions(int p, size_t q, const std::vector<rd_event_t> &events, ActionLists &out);

}  // namespace rd
#endif
