// From a schedule's send/receive pairs to what the kernels execute.
//
// Tree mode: per segment the pairs define one binary expression over the p inputs ("the receiving
// processor combines its segment with the segment received", Section IV).  The expression is built
// by replaying the pairs symbolically, then flattened into a program for a one-accumulator stack
// machine; operand roles (held / incoming) are kept in every operation so the evaluation order can
// be chosen freely (deepest subtree first, which keeps the stack at most log2 p deep).
//
// Faithful mode: per process the ordered list of its own sends and receives.
#include <algorithm>
#include <cstring>
#include <string>
#include <unordered_map>

#include "rd_internal.h"

namespace rd {

namespace {

struct Node { int32_t held, incoming; };   // children; ids < p are the processes' own data

struct Flattener {
    int p;
    const std::vector<Node> &nodes;        // nodes[k] is expression p + k
    const std::vector<int> &need;          // stack entries needed to evaluate expression id
    std::vector<uint32_t> &ops;

    bool leaf(int id) const { return id < p; }
    void emit(uint32_t kind, int proc) { ops.push_back(uint32_t(proc) | (kind << kIdxBits)); }
    int addPop(bool poppedIsHeld)
    {
        uint32_t &w = ops.back();
        const uint32_t n = (w >> (kIdxBits + 2)) & 0xF;
        if (n >= uint32_t(kMaxPops)) return RD_ERR_INTERNAL;
        if (poppedIsHeld) w |= uint32_t(1) << (kIdxBits + 6 + n);
        w = (w & ~(uint32_t(0xF) << (kIdxBits + 2))) | ((n + 1) << (kIdxBits + 2));
        return RD_OK;
    }
    int gen(int id, bool pushFirst)
    {
        if (leaf(id)) { emit(pushFirst ? OP_PUSH_LOAD : OP_LOAD, id); return RD_OK; }
        const Node &n = nodes[size_t(id - p)];
        if (leaf(n.held) && leaf(n.incoming)) {
            emit(pushFirst ? OP_PUSH_LOAD : OP_LOAD, n.held);
            emit(OP_ACC_IN, n.incoming);
            return RD_OK;
        }
        if (leaf(n.incoming)) {
            if (int rc = gen(n.held, pushFirst)) return rc;
            emit(OP_ACC_IN, n.incoming);
            return RD_OK;
        }
        if (leaf(n.held)) {
            if (int rc = gen(n.incoming, pushFirst)) return rc;
            emit(OP_ACC_HELD, n.held);
            return RD_OK;
        }
        const bool heldFirst = need[size_t(n.held)] >= need[size_t(n.incoming)];
        if (int rc = gen(heldFirst ? n.held : n.incoming, pushFirst)) return rc;
        if (int rc = gen(heldFirst ? n.incoming : n.held, true)) return rc;
        return addPop(heldFirst);
    }
};

}  // namespace

int compile_programs(int p, size_t q, const std::vector<rd_event_t> &events, Programs &out)
{
    if (p < 1 || p > kMaxProcs) return RD_ERR_INVALID_ARG;
    out.ops.clear();
    out.seg_prog.assign(q, 0);
    out.stack_depth = 0;
    out.shared_depth = 0;
    out.shared_pushes = 0;
    out.n_distinct = 0;
    // bucket the pairs by segment, keeping their start-time order
    std::vector<size_t> first(q + 1, 0);
    for (const rd_event_t &e : events) {
        if (e.seg < 0 || size_t(e.seg) >= q) return RD_ERR_INTERNAL;
        first[size_t(e.seg) + 1]++;
    }
    for (size_t j = 0; j < q; j++) first[j + 1] += first[j];
    std::vector<rd_event_t> bySeg(events.size());
    {
        std::vector<size_t> fill(first.begin(), first.end() - 1);
        for (const rd_event_t &e : events) bySeg[fill[size_t(e.seg)]++] = e;
    }
    std::unordered_map<std::string, uint32_t> seen;
    std::vector<Node> nodes;
    const size_t P = size_t(p);
    std::vector<int> expr(P, 0), need, leafSeen(P, 0);
    std::vector<uint32_t> prog;
    std::vector<int> walk;
    size_t pushedBefore = 0;                 // pushes that remain in the segment before this one
    for (size_t j = 0; j < q; j++) {
        // The program depends only on who sends to whom, in which order: a segment whose pairs repeat those of the
        // segment before it (every segment of a fixed tree, most segments of a greedy schedule's steady state)
        // shares that segment's program.
        if (j > 0 && first[j + 1] - first[j] == first[j] - first[j - 1]) {
            bool same = true;
            for (size_t k = first[j], k0 = first[j - 1]; k < first[j + 1] && same; k++, k0++)
                same = bySeg[k].src == bySeg[k0].src && bySeg[k].dst == bySeg[k0].dst && bySeg[k].kind == bySeg[k0].kind;
            if (same) {
                out.seg_prog[j] = out.seg_prog[j - 1];
                out.shared_pushes += pushedBefore;
                continue;
            }
        }
        nodes.clear();
        for (int i = 0; i < p; i++) expr[size_t(i)] = i;
        for (size_t k = first[j]; k < first[j + 1]; k++) {
            const rd_event_t &e = bySeg[k];
            if (e.src < 0 || e.src >= p || e.dst < 0 || e.dst >= p || e.src == e.dst) return RD_ERR_INTERNAL;
            if (e.kind == 0) {
                nodes.push_back(Node{expr[size_t(e.dst)], expr[size_t(e.src)]});
                expr[size_t(e.dst)] = p + int(nodes.size()) - 1;
            } else {
                expr[size_t(e.dst)] = expr[size_t(e.src)];
            }
        }
        const int root = expr[0];
        // every process's data must enter the root's expression exactly once
        std::fill(leafSeen.begin(), leafSeen.end(), 0);
        walk.assign(1, root);
        size_t leaves = 0;
        while (!walk.empty()) {
            const int id = walk.back(); walk.pop_back();
            if (id < p) { if (leafSeen[size_t(id)]++) return RD_ERR_INTERNAL; leaves++; continue; }
            walk.push_back(nodes[size_t(id - p)].held);
            walk.push_back(nodes[size_t(id - p)].incoming);
            if (leaves + walk.size() > size_t(2 * p)) return RD_ERR_INTERNAL;
        }
        if (leaves != size_t(p)) return RD_ERR_INTERNAL;
        // stack need, children before parents (a node only refers to older expressions)
        need.assign(size_t(p) + nodes.size(), 0);
        for (size_t k = 0; k < nodes.size(); k++) {
            const Node &n = nodes[k];
            const bool lh = n.held < p, li = n.incoming < p;
            int v;
            if (lh && li) v = 0;
            else if (li) v = need[size_t(n.held)];
            else if (lh) v = need[size_t(n.incoming)];
            else {
                const int a = std::max(need[size_t(n.held)], need[size_t(n.incoming)]);
                const int b = std::min(need[size_t(n.held)], need[size_t(n.incoming)]);
                v = std::max(a, b + 1);
            }
            need[size_t(p) + k] = v;
        }
        prog.clear();
        Flattener fl{p, nodes, need, prog};
        if (int rc = fl.gen(root, false)) return rc;
        if (prog.size() != size_t(p)) return RD_ERR_INTERNAL;
        if (need[size_t(root)] > kMaxPops) return RD_ERR_INTERNAL;
        out.stack_depth = std::max(out.stack_depth, need[size_t(root)]);
        // A pushed value that is popped again before anything else is pushed never has another entry above it,
        // and the sub-expression evaluated in between (the PUSH_LOAD, the combines that follow it, up to the
        // operation whose first pop takes the entry back) needs no stack of its own: a kernel may evaluate it in a
        // second accumulator and leave the running value where it is, instead of pushing and popping it.  Those
        // operations are marked, and so is the one that ends the sub-expression; what remains is the depth a
        // stack really needs then.
        {
            std::vector<std::pair<size_t, bool>> open;      // pushes not yet popped: (operation, still nothing above it)
            int onStack = 0, deepest = 0;
            size_t pushed = 0;                               // pushes that stay pushes
            for (size_t k = 0; k < prog.size(); k++) {
                if (((prog[k] >> kIdxBits) & 3u) == OP_PUSH_LOAD) {
                    if (!open.empty() && open.back().second) { open.back().second = false; deepest = std::max(deepest, ++onStack); }
                    open.emplace_back(k, true);
                }
                const uint32_t pops = (prog[k] >> (kIdxBits + 2)) & 0xFu;
                for (uint32_t m = 0; m < pops; m++) {
                    if (open.empty()) return RD_ERR_INTERNAL;
                    if (open.back().second) {
                        if (m != 0) return RD_ERR_INTERNAL;
                        for (size_t t = open.back().first; t <= k; t++) prog[t] |= kOpSecondAccumulator;
                        prog[k] |= kOpMergeSecond;
                    } else {
                        onStack--;
                        pushed++;
                    }
                    open.pop_back();
                }
            }
            if (!open.empty() || onStack != 0) return RD_ERR_INTERNAL;
            out.shared_depth = std::max(out.shared_depth, deepest);
            out.shared_pushes += pushed;
            pushedBefore = pushed;
        }
        std::string key(reinterpret_cast<const char *>(prog.data()), prog.size() * sizeof(uint32_t));
        auto it = seen.find(key);
        if (it == seen.end()) {
            it = seen.emplace(std::move(key), uint32_t(out.ops.size())).first;
            out.ops.insert(out.ops.end(), prog.begin(), prog.end());
            out.n_distinct++;
        }
        out.seg_prog[j] = it->second;
    }
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// Schedule-faithful execution: every process gets the list of its own sends and receives in
// start-time order (a send before a receive that starts at the same tick: with two ports a send
// is only a posting).  A process keeps its partial result of a segment in a scratch slot from its
// first receive of the segment until the send of that segment has been taken by the receiver;
// slots are recycled first-freed-first once the freeing send lies in the past of the schedule, and
// a receive into a recycled slot names the send whose completion it has to see first.  The root accumulates straight into the output buffer.
// ---------------------------------------------------------------------------------------------
int build_actions(int p, size_t q, const std::vector<rd_event_t> &events, ActionLists &out)
{
    const size_t P = size_t(p);
    out.actions.clear();
    out.first.assign(P + 1, 0);
    out.slots_per_proc = 0;
    for (const rd_event_t &e : events) { out.first[size_t(e.src) + 1]++; out.first[size_t(e.dst) + 1]++; }
    for (size_t i = 0; i < P; i++) out.first[i + 1] += out.first[i];
    out.actions.resize(out.first[P]);
    // events are ordered by start time; two passes keep "sends first" among equal times
    std::vector<uint32_t> fill(out.first.begin(), out.first.end() - 1);
    for (size_t k = 0; k < events.size();) {
        size_t k1 = k;
        while (k1 < events.size() && events[k1].t_start == events[k].t_start) k1++;
        for (size_t e = k; e < k1; e++) {
            Action a{events[e].seg, events[e].dst, 2, -1, -1, 0, int32_t(e), -1};
            out.actions[fill[size_t(events[e].src)]++] = a;
        }
        for (size_t e = k; e < k1; e++) {
            Action a{events[e].seg, events[e].src, events[e].kind == 0 ? 0 : 1, -1, -1, 0, int32_t(e), -1};
            out.actions[fill[size_t(events[e].dst)]++] = a;
        }
        k = k1;
    }
    // slots, process by process
    std::vector<int32_t> senderSlot(events.size(), -1);
    std::vector<int32_t> cur(q), arrivals(q);
    std::vector<std::pair<int32_t, int32_t>> freed;     // (slot, send that must be taken), oldest first
    for (size_t i = 0; i < P; i++) {
        std::fill(cur.begin(), cur.end(), -1);
        std::fill(arrivals.begin(), arrivals.end(), 0);
        freed.clear();
        size_t freedHead = 0;
        int used = 0;
        for (uint32_t k = out.first[i]; k < out.first[i + 1]; k++) {
            Action &a = out.actions[k];
            const size_t j = size_t(a.seg);
            if (a.kind == 2) {
                a.slot = i == 0 ? -2 : cur[j];
                if (i == 0 && arrivals[j] == 0) a.slot = -1;          // the root forwards its own input
                senderSlot[size_t(a.event)] = a.slot;
                if (a.slot >= 0) { freed.push_back(std::make_pair(a.slot, a.event)); cur[j] = -1; }
                arrivals[j] = 0;
            } else {
                a.first = arrivals[j] == 0 ? 1 : 0;
                arrivals[j]++;
                if (i == 0) { a.slot = -2; continue; }
                if (cur[j] < 0) {
                    // recycle only a slot whose send started earlier than this receive: the schedule
                    // itself then expects it to be over; otherwise take a fresh one
                    if (freedHead < freed.size() &&
                        events[size_t(freed[freedHead].second)].t_start < events[size_t(a.event)].t_start) {
                        cur[j] = freed[freedHead].first; a.wait_event = freed[freedHead].second; freedHead++;
                    } else cur[j] = used++;
                }
                a.slot = cur[j];
            }
        }
        out.slots_per_proc = std::max(out.slots_per_proc, used);
    }
    for (Action &a : out.actions)
        if (a.kind != 2) a.peer_slot = senderSlot[size_t(a.event)];
    return RD_OK;
}

}  // namespace rd
