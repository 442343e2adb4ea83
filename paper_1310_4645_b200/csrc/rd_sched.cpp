// Schedule generation (host): who sends which segment to whom, and when, under the
// linear model in integer ticks.  Times are exact, ties are broken by
// (time, process index) ascending.
#include <algorithm>
#include <cmath>
#include <functional>
#include <queue>
#include <utility>

#include "rd_internal.h"

namespace rd {

int ceil_log2(uint64_t v)
{
    int l = 0;
    while ((uint64_t(1) << l) < v) l++;
    return l;
}

void sort_events(std::vector<rd_event_t> &ev)
{
    std::sort(ev.begin(), ev.end(), [](const rd_event_t &a, const rd_event_t &b) {
        if (a.t_start != b.t_start) return a.t_start < b.t_start;
        if (a.seg != b.seg) return a.seg < b.seg;
        if (a.src != b.src) return a.src < b.src;
        return a.dst < b.dst;
    });
}

static bool event_before(const rd_event_t &a, const rd_event_t &b)
{
    if (a.t_start != b.t_start) return a.t_start < b.t_start;
    if (a.seg != b.seg) return a.seg < b.seg;
    if (a.src != b.src) return a.src < b.src;
    return a.dst < b.dst;
}

// Lock-step schedules: every pair starts at a multiple of the round length, and the generators emit the pairs
// segment by segment, process by process, so a stable counting sort on the round leaves each round in
// (segment, source) order: linear time where the comparison sort of a few million pairs takes longer than everything
// else together.  Falls back to the comparison sort when the rounds are too sparse or the order is not reached.
static void order_by_round(std::vector<rd_event_t> &ev, int64_t len)
{
    if (ev.size() < 2) return;
    if (std::is_sorted(ev.begin(), ev.end(), event_before)) return;
    int64_t last = -1;
    if (len > 0) {
        last = 0;
        for (const rd_event_t &e : ev) last = std::max(last, e.t_start / len);
    }
    if (last < 0 || uint64_t(last) > 8 * uint64_t(ev.size()) + 1024) { sort_events(ev); return; }
    std::vector<size_t> first(size_t(last) + 2, 0);
    for (const rd_event_t &e : ev) first[size_t(e.t_start / len) + 1]++;
    for (size_t r = 0; r + 1 < first.size(); r++) first[r + 1] += first[r];
    std::vector<rd_event_t> sorted(ev.size());
    for (const rd_event_t &e : ev) sorted[first[size_t(e.t_start / len)]++] = e;
    ev.swap(sorted);
    if (!std::is_sorted(ev.begin(), ev.end(), event_before)) sort_events(ev);
}

static void set_offsets(const std::vector<int64_t> &seg_bytes, Schedule &out)
{
    out.seg_off.assign(1, 0);
    for (int64_t b : seg_bytes) out.seg_off.push_back(out.seg_off.back() + uint64_t(b) / 4);
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1 (uni-greedy).  Per segment the two processes with the smallest states (ties: the smaller
// process index) among those that still hold the segment are paired at t = the larger of the two states;
// the root never sends (Lemma 1), so it is the receiver whenever it is one of the two.
// The pairing instants of a segment never decrease, so the receivers' new states come out in
// non-decreasing order: as in the two-queue construction of a Huffman tree, the smallest state is always
// at the head of one of two sorted queues (the states the segment started with; the states of receivers),
// and a segment costs O(p) once its initial states are in order.  They are: the senders' states after a
// segment, taken in pairing order, are sorted already, and the root, the last receiver, has the largest.
// Equal states are put in process order where they meet (runs of equal states are short).
// ---------------------------------------------------------------------------------------------
int gen_uni_greedy(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, Schedule &out, bool want_events)
{
    typedef std::pair<int64_t, int> Key;                 // (state, process)
    out.events.clear();
    out.completion = 0;
    set_offsets(seg_bytes, out);
    if (p < 1) return RD_OK;
    if (want_events) out.events.reserve(size_t(p - 1) * seg_bytes.size());
    std::vector<Key> start, next, received;
    for (int i = 0; i < p; i++) start.push_back(Key(0, i));
    for (size_t j = 0; j < seg_bytes.size(); j++) {
        const int64_t tc = c.comm(seg_bytes[j]), tp = c.comp(seg_bytes[j]);
        size_t h1 = 0, h2 = 0;
        received.clear();
        next.clear();
        auto take = [&]() {
            if (h1 < start.size() && (h2 >= received.size() || start[h1] < received[h2])) return start[h1++];
            return received[h2++];
        };
        for (int k = 0; k + 1 < p; k++) {
            const Key first = take(), second = take();
            const int64_t t = second.first;
            int sender = first.second, receiver = second.second;
            if (sender == 0) std::swap(sender, receiver);
            if (want_events) out.events.push_back(rd_event_t{int32_t(j), sender, receiver, 0, t});
            next.push_back(Key(t + tc, sender));
            // no state in the queue is larger than the new one: it joins the run of equal states at the end
            const Key key(t + tc + tp, receiver);
            received.insert(std::upper_bound(received.begin() + std::ptrdiff_t(h2), received.end(), key), key);
        }
        next.push_back(take());                          // the root, with the largest state
        for (size_t a = 0; a < next.size();) {           // runs of equal states in process order
            size_t b = a + 1;
            while (b < next.size() && next[b].first == next[a].first) b++;
            if (b - a > 1) std::sort(next.begin() + std::ptrdiff_t(a), next.begin() + std::ptrdiff_t(b));
            a = b;
        }
        start.swap(next);
    }
    for (const Key &k : start)
        if (k.second == 0) out.completion = k.first;
    if (want_events) sort_events(out.events);
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// Algorithm 2 (bi-greedy), event driven.  At every instant a port frees, segments are visited in
// increasing index starting with the first the root has not completed; for each, the processes
// able to send it and those able to receive it are matched entry-wise in process order, the ones
// free in both directions being dealt to whichever side is short (front of the list receives, back
// of the list sends).  A process is skipped while a communication of the segment's length would
// run into its scheduled combine; a combine waits for a send of the same process still running.
// ---------------------------------------------------------------------------------------------
int gen_bi_greedy(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, Schedule &out, bool want_events)
{
    const size_t q = seg_bytes.size();
    out.events.clear();
    set_offsets(seg_bytes, out);
    out.completion = 0;
    if (p < 2 || q == 0) return RD_OK;
    const size_t P = size_t(p);
    std::vector<int64_t> sendFreeAt(P, 0), recvFreeAt(P, 0), compBegin(P, 0), compEnd(P, 0);
    std::vector<uint8_t> sent(P * q, 0);              // sent[i*q + j]: i has sent j (root: j complete)
    std::vector<int64_t> lastSendEnd(q, 0);
    std::vector<uint32_t> holders(q, uint32_t(p));    // processes (root included) not yet done with j
    std::vector<int> sendOnly, recvOnly, both, sendList, recvList, idle;
    std::vector<int64_t> fruitless;                   // segment lengths that cannot be paired at the current instant
    size_t rootNext = 0;                              // first segment the root has not completed
    int64_t t = 0;
    while (rootNext < q) {
        // the processes with a free port at this instant, in process order: only they can be paired now
        int freeSend = 0, freeRecv = 0, freeSendNonRoot = 0;
        idle.clear();
        fruitless.clear();
        for (int i = 0; i < p; i++) {
            const bool s = sendFreeAt[size_t(i)] <= t, r = recvFreeAt[size_t(i)] <= t;
            if (s) { freeSend++; if (i != 0) freeSendNonRoot++; }
            if (r) freeRecv++;
            if ((s && i != 0) || r) idle.push_back(i);
        }
        for (size_t j = rootNext; j < q; j++) {
            if (freeSendNonRoot == 0 || freeRecv == 0) break;   // nothing can be paired from here on
            // A segment that none of the idle processes has sent yet and that still found no pair (ports free on one
            // side only, or combines in the way) settles every later segment of its length at this instant: their
            // candidates are a subset of its, and fewer candidates never make a pair where more made none.
            if (std::find(fruitless.begin(), fruitless.end(), seg_bytes[j]) != fruitless.end()) continue;
            const int64_t tc = c.comm(seg_bytes[j]), tp = c.comp(seg_bytes[j]);
            sendOnly.clear(); recvOnly.clear(); both.clear();
            bool allHold = true;
            for (int i : idle) {
                const size_t I = size_t(i);
                if (sent[I * q + j]) { allHold = false; continue; }
                if (t < compEnd[I] && compBegin[I] < t + tc) continue;        // would meet its combine
                const bool canSend = i != 0 && sendFreeAt[I] <= t;
                const bool canRecv = recvFreeAt[I] <= t;
                if (canSend && canRecv) both.push_back(i);
                else if (canSend) sendOnly.push_back(i);
                else if (canRecv) recvOnly.push_back(i);
            }
            const int s = int(sendOnly.size()), r = int(recvOnly.size()), f = int(both.size());
            int toRecv = 0, toSend = 0;               // prefix of `both` that receives, suffix that sends
            if (s == r) { toRecv = toSend = f / 2; }
            else if (s < r) { const int m = std::min(f, r - s), x = (f - m) / 2; toSend = m > 0 ? m + x : 0; toRecv = x; }
            else { const int m = std::min(f, s - r), x = (f - m) / 2; toRecv = m > 0 ? m + x : 0; toSend = x; }
            // when m = 0 the short side gets nothing extra; x may still be positive on the other branch
            if (s < r && std::min(f, r - s) == 0) toSend = 0;
            if (s > r && std::min(f, s - r) == 0) toRecv = 0;
            sendList.assign(sendOnly.begin(), sendOnly.end());
            sendList.insert(sendList.end(), both.end() - toSend, both.end());
            std::sort(sendList.begin(), sendList.end());
            recvList.assign(recvOnly.begin(), recvOnly.end());
            recvList.insert(recvList.end(), both.begin(), both.begin() + toRecv);
            std::sort(recvList.begin(), recvList.end());
            const size_t pairs = std::min(sendList.size(), recvList.size());
            if (pairs == 0 && allHold) fruitless.push_back(seg_bytes[j]);
            for (size_t k = 0; k < pairs; k++) {
                const int a = sendList[k], b = recvList[k];
                const size_t Ia = size_t(a), Ib = size_t(b);
                sent[Ia * q + j] = 1; holders[j]--;
                sendFreeAt[Ia] = t + tc;
                if (t + tc > lastSendEnd[j]) lastSendEnd[j] = t + tc;
                int64_t begin = t + tc;
                if (tp > 0 && sendFreeAt[Ib] > begin) begin = sendFreeAt[Ib];
                compBegin[Ib] = begin; compEnd[Ib] = begin + tp; recvFreeAt[Ib] = begin + tp;
                if (want_events) out.events.push_back(rd_event_t{int32_t(j), a, b, 0, t});
                freeSend--; freeSendNonRoot--; freeRecv--;
            }
            if (holders[j] == 1 && !sent[0 * q + j]) {            // only the root is left: segment complete
                sent[0 * q + j] = 1; holders[j] = 0;
                const int64_t done = lastSendEnd[j] + tp;
                if (done > out.completion) out.completion = done;
            }
            if (freeSend + freeRecv < 2) break;
        }
        while (rootNext < q && sent[0 * q + rootNext]) rootNext++;
        if (rootNext >= q) break;
        int64_t next = -1;
        for (int i = 0; i < p; i++) {
            const int64_t a = sendFreeAt[size_t(i)], b = recvFreeAt[size_t(i)];
            if (a > t && (next < 0 || a < next)) next = a;
            if (b > t && (next < 0 || b < next)) next = b;
        }
        if (next < 0) return RD_ERR_INTERNAL;
        t = next;
    }
    if (want_events) sort_events(out.events);
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// Section IV, lock-step rounds of length alpha + (beta + gamma) * s with s the full segment size.
// ---------------------------------------------------------------------------------------------
static int64_t round_length(const std::vector<int64_t> &seg_bytes, const Ticks &c)
{
    int64_t s = 0;
    for (int64_t b : seg_bytes) s = std::max(s, b);
    return c.comm(s) + c.comp(s);
}

int gen_binomial(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, Schedule &out)
{
    const int rounds = ceil_log2(uint64_t(p));
    const int64_t len = round_length(seg_bytes, c);
    out.events.clear();
    out.events.reserve(size_t(p > 0 ? p - 1 : 0) * seg_bytes.size());
    for (size_t j = 0; j < seg_bytes.size(); j++)
        for (int r = 0; r < rounds; r++)
            for (int64_t k = int64_t(1) << r; k < p; k += int64_t(2) << r)
                out.events.push_back(rd_event_t{int32_t(j), int32_t(k), int32_t(k - (int64_t(1) << r)), 0,
                                                (int64_t(j) * rounds + r) * len});
    out.completion = int64_t(seg_bytes.size()) * rounds * len;
    set_offsets(seg_bytes, out);
    order_by_round(out.events, len);
    return RD_OK;
}

int gen_pipeline(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, bool bidir, Schedule &out)
{
    const int64_t len = round_length(seg_bytes, c);
    const int64_t q = int64_t(seg_bytes.size());
    const int64_t perSegment = bidir ? 1 : 2;   // a one-port process alternates receive and send
    out.events.clear();
    out.completion = (p < 2 || q == 0) ? 0 : (int64_t(p - 1) + perSegment * (q - 1)) * len;
    set_offsets(seg_bytes, out);
    if (p < 2 || q == 0) return RD_OK;
    // process k sends segment j in round (p - 1 - k) + perSegment * j; emitted round by round, in a round by segment
    out.events.reserve(size_t(p - 1) * size_t(q));
    const int64_t lastRound = int64_t(p - 2) + perSegment * (q - 1);
    for (int64_t round = 0; round <= lastRound; round++) {
        const int64_t over = round - int64_t(p - 2);                         // segments before this one are through
        int64_t j = over > 0 ? (over + perSegment - 1) / perSegment : 0;
        for (; j < q && perSegment * j <= round; j++) {
            const int k = int(int64_t(p - 1) - (round - perSegment * j));
            out.events.push_back(rd_event_t{int32_t(j), k, k - 1, 0, round * len});
        }
    }
    return RD_OK;
}

int gen_binary(int p, const std::vector<int64_t> &seg_bytes, const Ticks &c, bool bidir, Schedule &out)
{
    const int64_t len = round_length(seg_bytes, c);
    const int64_t q = int64_t(seg_bytes.size());
    const int depth = ceil_log2(uint64_t(p) + 1) - 1;       // heap-ordered tree, root at depth 0
    const int64_t perSegment = bidir ? 2 : 4;
    int64_t rounds = 0;
    out.events.clear();
    out.events.reserve(size_t(p > 0 ? p - 1 : 0) * seg_bytes.size());
    for (int64_t j = 0; j < q; j++) {
        for (int k = 1; k < p; k++) {
            const int d = ceil_log2(uint64_t(k) + 2) - 1;    // depth of node k = floor(log2(k+1))
            const int64_t round = 2 * int64_t(depth - d) + ((k & 1) ? 0 : 1) + perSegment * j;   // left child first
            rounds = std::max(rounds, round + 1);
            out.events.push_back(rd_event_t{int32_t(j), k, (k - 1) / 2, 0, round * len});
        }
    }
    out.completion = rounds * len;
    set_offsets(seg_bytes, out);
    order_by_round(out.events, len);
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// Section III butterfly: recursive halving (distance p/2 first, the process with the distance bit
// clear keeps the lower half), then a binomial gather of the p reduced chunks to process 0.  When the
// number of processes is not a power of two, those beyond the largest power of two are folded into
// partners below it first (the improved algorithm the paper cites for that case is not described there).
// ---------------------------------------------------------------------------------------------
int gen_butterfly(int pAll, uint64_t n, const Ticks &c, Schedule &out)
{
    if (pAll < 1) return RD_ERR_INVALID_ARG;
    int p = 1;                                    // the largest power of two not above pAll
    while (2 * p <= pAll) p *= 2;
    const int L = ceil_log2(uint64_t(p));
    const size_t P = size_t(p);
    // chunk boundaries: follow each process's range through the halvings
    std::vector<uint64_t> lo(P, 0), hi(P, n);
    out.events.clear();
    int64_t t = 0;
    if (pAll > p) {
        // fold: every process beyond the power of two hands its whole message to a partner below it
        for (int i = 0; i < pAll - p; i++)
            for (int ch = 0; ch < p; ch++) out.events.push_back(rd_event_t{ch, p + i, i, 0, 0});
        t = c.comm(int64_t(n) * 4) + c.comp(int64_t(n) * 4);
    }
    for (int r = 0; r < L; r++) {
        const int d = p >> (r + 1);
        int64_t longest = 0;
        for (int k = 0; k < p; k++) {
            const uint64_t mid = lo[size_t(k)] + (hi[size_t(k)] - lo[size_t(k)]) / 2;
            const uint64_t keepLo = (k & d) ? mid : lo[size_t(k)], keepHi = (k & d) ? hi[size_t(k)] : mid;
            const int64_t bytes = int64_t(keepHi - keepLo) * 4;
            longest = std::max(longest, c.comm(bytes) + c.comp(bytes));
            const int firstChunk = k & ~(d - 1);               // chunks whose owner shares k's leading bits
            for (int ch = firstChunk; ch < firstChunk + d; ch++)
                out.events.push_back(rd_event_t{ch, k ^ d, k, 0, t});
        }
        for (int k = 0; k < p; k++) {
            const uint64_t mid = lo[size_t(k)] + (hi[size_t(k)] - lo[size_t(k)]) / 2;
            if (k & d) lo[size_t(k)] = mid; else hi[size_t(k)] = mid;
        }
        t += longest;
    }
    out.seg_off.resize(P + 1);
    for (int k = 0; k < p; k++) out.seg_off[size_t(k)] = lo[size_t(k)];
    out.seg_off[P] = n;
    for (int d = 1; d < p; d *= 2) {
        int64_t longest = 0;
        for (int k = d; k < p; k += 2 * d) {
            const int64_t bytes = int64_t(hi[size_t(k + d - 1)] - lo[size_t(k)]) * 4;
            longest = std::max(longest, c.comm(bytes));
            for (int ch = k; ch < k + d; ch++) out.events.push_back(rd_event_t{ch, k, k - d, 1, t});
        }
        t += longest;
    }
    out.completion = t;
    sort_events(out.events);
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// Segment size that minimises the completion time (Tables I and III; Section VII protocol).
// ---------------------------------------------------------------------------------------------
static std::vector<int64_t> equal_segments(size_t msg_bytes, size_t seg_bytes)
{
    std::vector<int64_t> v;
    for (size_t done = 0; done < msg_bytes; done += seg_bytes) v.push_back(int64_t(std::min(seg_bytes, msg_bytes - done)));
    return v;
}

int optimal_segment(rd_algo_t algo, rd_port_t port, int p, size_t m, const Ticks &c, size_t *out)
{
    if (m < 4) { *out = m; return RD_OK; }
    const bool bidir = port == RD_PORT_BI;
    if (algo == RD_BINOMIAL || algo == RD_BUTTERFLY || p < 2) { *out = m; return RD_OK; }
    if (algo == RD_UNI_GREEDY) {
        // powers of two from the largest down; stop once the time has risen twice in a row
        size_t best = m;
        Schedule tmp;
        gen_uni_greedy(p, equal_segments(m, m), c, tmp, false);
        int64_t bestT = tmp.completion, prev = bestT;
        int rises = 0;
        for (int i = ceil_log2(m) - ((size_t(1) << ceil_log2(m)) > m ? 1 : 0); i >= 2; i--) {
            const size_t s = size_t(1) << i;
            if (s >= m) continue;
            if ((m + s - 1) / s > (size_t(1) << 14)) break;
            gen_uni_greedy(p, equal_segments(m, s), c, tmp, false);
            if (tmp.completion < bestT) { bestT = tmp.completion; best = s; }
            rises = tmp.completion > prev ? rises + 1 : 0;
            prev = tmp.completion;
            if (rises >= 2) break;
        }
        *out = best;
        return RD_OK;
    }
    // closed forms: rounds(q) * (alpha + (beta+gamma) s), rounds(q) = lead + perSegment * (q - 1)
    double lead, perSegment, denomCount;
    const double N = double(ceil_log2(uint64_t(p) + 1));
    if (algo == RD_PIPELINE) { lead = p - 1; perSegment = bidir ? 1 : 2; denomCount = bidir ? p - 2 : p - 3; }
    else if (algo == RD_BINARY) { lead = 2 * (N - 1); perSegment = bidir ? 2 : 4; denomCount = bidir ? N - 2 : N - 3; }
    else if (algo == RD_BI_GREEDY) { lead = double(ceil_log2(uint64_t(p))); perSegment = 1; denomCount = lead - 1; }
    else return RD_ERR_INVALID_ARG;
    const double bg = double(c.B) + double(c.G);
    const double numer = (bidir || algo == RD_BI_GREEDY ? 1.0 : 2.0) * double(m) * double(c.A);
    if (denomCount <= 0 || bg <= 0) { *out = m; return RD_OK; }
    const double sOpt = std::sqrt(numer / (denomCount * bg));
    if (!(sOpt < double(m))) { *out = m; return RD_OK; }
    auto timeFor = [&](size_t s) {
        const double q = double((m + s - 1) / s);
        return (lead + perSegment * (q - 1)) * (double(c.A) + bg * double(s));
    };
    auto segFor = [&](size_t q) {               // equal segments for q pieces, multiple of 4 bytes
        size_t s = (m + q - 1) / q;
        s = (s + 3) / 4 * 4;
        return std::max<size_t>(4, std::min(s, m));
    };
    const double qReal = sOpt > 0 ? double(m) / sOpt : double(m) / 4;
    size_t qLo = size_t(std::max(1.0, std::floor(qReal))), qHi = size_t(std::max(1.0, std::ceil(qReal)));
    qLo = std::min(qLo, m / 4); qHi = std::min(qHi, m / 4);
    const size_t sA = segFor(qLo), sB = segFor(qHi);     // sA >= sB
    *out = timeFor(sB) < timeFor(sA) ? sB : sA;
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// Section VIII: unequal segmentation for uni-greedy.  Start from the best equi-segmentation in
// multiples of `unit` bytes and move one unit at a time from one segment to another while that
// shortens the completion time (the paper observes that the optimum is usually one or two such moves
// away from the best equi-segmentation).
// ---------------------------------------------------------------------------------------------
static void neighbours(const std::vector<int64_t> &seg, int64_t unit, std::vector<std::vector<int64_t>> &out)
{
    for (size_t i = 0; i < seg.size(); i++) {
        for (size_t j = 0; j < seg.size(); j++) {              // one unit from segment i to segment j
            if (i == j) continue;
            std::vector<int64_t> v = seg;
            v[i] -= unit; v[j] += unit;
            if (v[i] == 0) v.erase(v.begin() + long(i));
            out.push_back(std::move(v));
        }
        if (seg[i] > unit) {                                   // one unit split off into a new last segment
            std::vector<int64_t> v = seg;
            v[i] -= unit; v.push_back(unit);
            out.push_back(std::move(v));
        }
    }
}

int search_segmentation(int p, size_t msg_bytes, size_t unit, const Ticks &c, std::vector<int64_t> &best, int64_t *bestTicks)
{
    if (unit == 0 || (unit & 3u) || msg_bytes == 0 || msg_bytes % unit) return RD_ERR_INVALID_ARG;
    const size_t units = msg_bytes / unit;
    if (units > 4096) return RD_ERR_INVALID_ARG;
    Schedule tmp;
    auto timeOf = [&](const std::vector<int64_t> &seg) { gen_uni_greedy(p, seg, c, tmp, false); return tmp.completion; };
    // every equi-segmentation (k units per segment) that reaches the best equi time is a starting point
    std::vector<std::vector<int64_t>> starts;
    int64_t equiT = -1;
    for (size_t k = 1; k <= units; k++) {
        std::vector<int64_t> seg = equal_segments(msg_bytes, k * unit);
        const int64_t t = timeOf(seg);
        if (equiT < 0 || t < equiT) { equiT = t; starts.clear(); }
        if (t == equiT) starts.push_back(std::move(seg));
    }
    int64_t bestT = equiT;
    best = starts.front();
    std::vector<std::vector<int64_t>> near, far;
    for (const std::vector<int64_t> &start : starts) {
        std::vector<int64_t> cur = start;
        int64_t curT = equiT;
        for (bool improved = true; improved;) {
            improved = false;
            near.clear();
            neighbours(cur, int64_t(unit), near);
            std::vector<int64_t> pick;
            int64_t pickT = curT;
            for (const std::vector<int64_t> &v : near) {
                const int64_t t = timeOf(v);
                if (t < pickT) { pickT = t; pick = v; }
            }
            if (pickT == curT && near.size() * near.size() <= 40000) {     // nothing one move away: look two moves away
                for (const std::vector<int64_t> &v : near) {
                    far.clear();
                    neighbours(v, int64_t(unit), far);
                    for (const std::vector<int64_t> &w : far) {
                        const int64_t t = timeOf(w);
                        if (t < pickT) { pickT = t; pick = w; }
                    }
                }
            }
            if (pickT < curT) { curT = pickT; cur = pick; improved = true; }
        }
        if (curT < bestT) { bestT = curT; best = cur; }
    }
    *bestTicks = bestT;
    return RD_OK;
}

}  // namespace rd
