/*
 * rd_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, single-threaded CPU statement of what the pipelined-reduction
 * path computes, written from the paper (Lowery & Langou, "A Greedy Algorithm
 * for Optimally Pipelining a Reduction").  It is the authority the CUDA path
 * is compared with; it shares no code, header, table or helper with the
 * library and must never be linked into it or called from it.  Only tests,
 * the smoke check and the benchmark's CPU-baseline leg may use it.
 *
 * Two parts:
 *   O1  schedule simulators (Section IV, Algorithm 1, Algorithm 2, the
 *       reduce-scatter/gather of Section III) + a validity checker (Lemma 1,
 *       Section II port rules) + the "every contribution reaches the root
 *       exactly once" check (Section IV).
 *   O2  the reduction itself: per segment, replay the send/receive pairs in
 *       start-time order, the receiver combining what it holds with what it
 *       receives (Section IV, first paragraph).
 *
 * Time is an exact integer number of ticks: t_comm(j) = A + B*size(j),
 * t_comp(j) = G*size(j) (Section V, first paragraph), so that ties are decided
 * identically everywhere.
 *
 * Pins (tests/test_oracle_*.py): Table I and Table III closed forms, Table IV
 * (all 61 rows: ratio, best equi-segmentation, set of optimal segmentations),
 * the 61-of-986 census, the Fig. 8 makespan, the bi-greedy = reverse optimal
 * broadcast conjecture, Theorem 5 by brute force, Table II lower bounds, the
 * q = 1 special case, order-free integer results.
 *
 * Parity unpinned: WHICH processes pair with which in bi-greedy beyond what
 * the completion time, the validity rules and the contribution invariant fix
 * (the figure that shows the pairing is not available); the same holds for
 * uni-greedy process identities (only the makespan of the Fig. 3 example is
 * checkable).  The tie-break used is (time, process index) ascending.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC.  A second build of the same file
 * with -fopenmp added lets several threads share the int32 and fp32 evaluators: every thread replays
 * all the events on its own range of the elements of each segment (an element's result depends on
 * that element of the p inputs only), so the arithmetic per element is the same and so are the bits.
 * It exists so that the benchmark can time the oracle on all host cores; parity tests use the plain build.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t seg;     /* segment index, 0-based (butterfly: final chunk index)      */
    int32_t src;     /* sending process                                          */
    int32_t dst;     /* receiving process                                        */
    int32_t kind;    /* 0 = receiver combines, 1 = receiver only stores (gather) */
    int64_t t_start; /* tick at which the communication starts                   */
} orc_event_t;

enum { ORC_OK = 0, ORC_BAD_ARG = -1, ORC_STUCK = -2, ORC_NOMEM = -3 };

/* ------------------------------------------------------------------------- */
/* Cost model, Section II (Hockney) and Section V: t_comm = alpha + beta*s,  */
/* t_comp = gamma*s, in integer ticks.                                       */
/* ------------------------------------------------------------------------- */
static int64_t t_comm(int64_t A, int64_t B, int64_t size) { return A + B * size; }
static int64_t t_comp(int64_t G, int64_t size) { return G * size; }

int orc_ceil_log2(int64_t v)
{
    int l = 0;
    int64_t x = 1;
    while (x < v) { x *= 2; l++; }
    return l;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1 (uni-greedy).  State x[i] = time process i finished its last  */
/* task.  Per segment, while more than one process remains: order the        */
/* remaining states, take the two smallest g1, g2, start at t = x[g2]        */
/* (Lemma 1 (iii) with equality).  The root may not send (Lemma 1 (ii)), so  */
/* when g1 is the root g2 sends to it; otherwise g1 sends to g2.  Sender is  */
/* free at t + t_comm, receiver at t + t_comm + t_comp; the final states of  */
/* one segment start the next.  Ties: (time, index) ascending.               */
/* sizes[j] is the size of segment j in the unit B and G are expressed in.   */
/* events may be NULL (time only).  Returns completion = final root state.   */
/* ------------------------------------------------------------------------- */
int orc_uni_greedy(int p, int q, const int64_t *sizes, int64_t A, int64_t B, int64_t G,
                   orc_event_t *events, int64_t *completion)
{
    if (p < 1 || q < 1 || !sizes) return ORC_BAD_ARG;
    int64_t *x = (int64_t *)calloc((size_t)p, sizeof(int64_t));
    int *I = (int *)malloc(sizeof(int) * (size_t)p);             /* processes that still hold segment j, ascending */
    int64_t *X = (int64_t *)malloc(sizeof(int64_t) * (size_t)p); /* their states, X[k] = x[I[k]]                   */
    if (!x || !I || !X) { free(x); free(I); free(X); return ORC_NOMEM; }
    size_t ne = 0;
    for (int j = 0; j < q; j++) {
        int64_t tc = t_comm(A, B, sizes[j]), tp = t_comp(G, sizes[j]);
        for (int i = 0; i < p; i++) { I[i] = i; X[i] = x[i]; }
        for (int left = p; left >= 2; left--) {
            int k1 = 0, k2 = -1;                    /* positions of the smallest and second smallest state */
            for (int k = 1; k < left; k++) {
                if (X[k] < X[k1]) { k2 = k1; k1 = k; }
                else if (k2 < 0 || X[k] < X[k2]) { k2 = k; }
            }
            int64_t t = X[k2];
            int ka = k1, kb = k2;                   /* sender, receiver */
            if (I[ka] == 0) { ka = k2; kb = k1; }
            int a = I[ka], b = I[kb];
            if (events) {
                events[ne].seg = j; events[ne].src = a; events[ne].dst = b;
                events[ne].kind = 0; events[ne].t_start = t;
            }
            ne++;
            x[a] = t + tc;
            x[b] = X[kb] = t + tc + tp;
            memmove(&I[ka], &I[ka + 1], sizeof(int) * (size_t)(left - 1 - ka));       /* a has sent segment j */
            memmove(&X[ka], &X[ka + 1], sizeof(int64_t) * (size_t)(left - 1 - ka));
        }
    }
    if (completion) *completion = x[0];
    free(x); free(I); free(X);
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2 (bi-greedy).  Arrays as in the paper: S, R = time the send /  */
/* receive port of a process is free again; C1, C2 = start and end of its    */
/* last scheduled computation; M(i,j) = time process i finished sending      */
/* segment j (root: time the segment is complete).  "sent" replaces the      */
/* paper's M = 0 sentinel.                                                   */
/* Readings: a process is in COMP when the would-be communication            */
/* [t, t+t_comm(j)) meets its scheduled computation (t < C2 and              */
/* C1 < t + t_comm(j)); the combination of a received segment waits for a    */
/* send of the same process that is still running (Section II:               */
/* communication and computation do not overlap; only a smaller last segment */
/* can trigger this); the root is never a sender; every set is               */
/* kept in ascending process order and paired entry-wise; time advances to   */
/* the next instant a port frees (unit_step = 0) or by 1 as printed          */
/* (unit_step = 1).                                                          */
/* ------------------------------------------------------------------------- */
int orc_bi_greedy(int p, int q, const int64_t *sizes, int64_t A, int64_t B, int64_t G,
                  int unit_step, orc_event_t *events, int64_t *completion)
{
    if (p < 1 || q < 1 || !sizes) return ORC_BAD_ARG;
    if (p == 1) { if (completion) *completion = 0; return ORC_OK; }   /* nothing to send */
    int64_t *S = calloc((size_t)p, 8), *R = calloc((size_t)p, 8);
    int64_t *C1 = calloc((size_t)p, 8), *C2 = calloc((size_t)p, 8);
    int64_t *M = calloc((size_t)p * (size_t)q, 8);
    char *sent = calloc((size_t)p * (size_t)q, 1);
    int *sendProc = malloc(sizeof(int) * (size_t)p), *recvProc = malloc(sizeof(int) * (size_t)p);
    int *freeProc = malloc(sizeof(int) * (size_t)p);
    char *inS = malloc((size_t)p), *inR = malloc((size_t)p);
    int rc = ORC_OK;
    size_t ne = 0;
    if (!S || !R || !C1 || !C2 || !M || !sent || !sendProc || !recvProc || !freeProc || !inS || !inR) {
        rc = ORC_NOMEM; goto done;
    }
    int64_t t = 0;
    size_t unsent = (size_t)p * (size_t)q;
    while (unsent > 0) {
        int segStart = 0;
        while (segStart < q && sent[0 * (size_t)q + segStart]) segStart++;
        if (segStart >= q) { rc = ORC_STUCK; goto done; }
        int stop = 1;
        int j = segStart - 1;
        while (stop) {
            j++;
            int64_t tc = t_comm(A, B, sizes[j]), tp = t_comp(G, sizes[j]);
            /* candidate sets */
            for (int i = 0; i < p; i++) {
                int inI = !sent[(size_t)i * q + j];
                int comp = (t < C2[i]) && (C1[i] < t + tc);
                inS[i] = (char)(inI && !comp && !(S[i] > t) && i != 0);
                inR[i] = (char)(inI && !comp && !(R[i] > t));
            }
            int s = 0, r = 0, f = 0;
            for (int i = 0; i < p; i++) {
                if (inS[i] && inR[i]) { freeProc[f++] = i; inS[i] = 0; inR[i] = 0; }
            }
            for (int i = 0; i < p; i++) { s += inS[i]; r += inR[i]; }
            /* hand the processes free in both directions to the two sides;
             * freeProc(k) below is 1-based as printed                        */
            if (s == r) {
                int y = f / 2;
                for (int k = f - y + 1; k <= f; k++) inS[freeProc[k - 1]] = 1;
                for (int k = 1; k <= y; k++) inR[freeProc[k - 1]] = 1;
            } else if (s < r) {
                int y = r - s;
                int m = f < y ? f : y;
                int xx = (f - m) / 2;
                if (m > 0) for (int k = f - (m + xx) + 1; k <= f; k++) inS[freeProc[k - 1]] = 1;
                if (xx > 0) for (int k = 1; k <= xx; k++) inR[freeProc[k - 1]] = 1;
            } else {
                int y = s - r;
                int m = f < y ? f : y;
                int xx = (f - m) / 2;
                if (m > 0) for (int k = 1; k <= m + xx; k++) inR[freeProc[k - 1]] = 1;
                if (xx > 0) for (int k = f - xx + 1; k <= f; k++) inS[freeProc[k - 1]] = 1;
            }
            int ns = 0, nr = 0;
            for (int i = 0; i < p; i++) {           /* ascending process order */
                if (inS[i]) sendProc[ns++] = i;
                if (inR[i]) recvProc[nr++] = i;
            }
            int l = ns < nr ? ns : nr;
            for (int k = 0; k < l; k++) {
                int a = sendProc[k], b = recvProc[k];
                M[(size_t)a * q + j] = t + tc;
                sent[(size_t)a * q + j] = 1; unsent--;
                S[a] = t + tc;
                /* the combination follows the receive, but waits for a send of the
                 * receiver that is still running (only a smaller last segment makes
                 * a receive end before a send that started no later)              */
                int64_t cs = t + tc;
                if (tp > 0 && S[b] > cs) cs = S[b];
                R[b] = cs + tp;
                C1[b] = cs;
                C2[b] = cs + tp;
                if (events) {
                    events[ne].seg = j; events[ne].src = a; events[ne].dst = b;
                    events[ne].kind = 0; events[ne].t_start = t;
                }
                ne++;
            }
            /* only the root is left for segment j: it completes after the
             * last arrival has been combined                                 */
            {
                int left = 0;
                for (int i = 0; i < p; i++) left += !sent[(size_t)i * q + j];
                if (left == 1 && !sent[0 * (size_t)q + j]) {
                    int64_t mx = 0;
                    for (int i = 0; i < p; i++) if (M[(size_t)i * q + j] > mx) mx = M[(size_t)i * q + j];
                    M[0 * (size_t)q + j] = mx + tp;
                    sent[0 * (size_t)q + j] = 1; unsent--;
                }
            }
            int freePorts = 0;
            for (int i = 0; i < p; i++) freePorts += (S[i] <= t) + (R[i] <= t);
            if (freePorts < 2) stop = 0;
            else if (j + 1 >= q) stop = 0;
        }
        if (unsent == 0) break;
        if (unit_step) {
            t = t + 1;
        } else {
            int64_t nxt = -1;
            for (int i = 0; i < p; i++) {
                if (S[i] > t && (nxt < 0 || S[i] < nxt)) nxt = S[i];
                if (R[i] > t && (nxt < 0 || R[i] < nxt)) nxt = R[i];
            }
            if (nxt < 0) { rc = ORC_STUCK; goto done; }
            t = nxt;
        }
    }
    if (completion) {
        int64_t mx = 0;
        for (int j = 0; j < q; j++) if (M[j] > mx) mx = M[j];
        *completion = mx;
    }
done:
    free(S); free(R); free(C1); free(C2); free(M); free(sent);
    free(sendProc); free(recvProc); free(freeProc); free(inS); free(inR);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* The three standard algorithms of Section IV as lock-step rounds of length */
/* alpha + beta*s + gamma*s (s = the largest segment, i.e. the full segment  */
/* size of an equi-segmentation), which is how Tables I and III count them.  */
/* bidir = 0: unidirectional ports.                                          */
/* ------------------------------------------------------------------------- */
static int64_t round_length(int q, const int64_t *sizes, int64_t A, int64_t B, int64_t G)
{
    int64_t s = 0;
    for (int j = 0; j < q; j++) if (sizes[j] > s) s = sizes[j];
    return t_comm(A, B, s) + t_comp(G, s);
}

/* Binomial: with n processes left, floor(n/2) send and floor(n/2) receive,
 * ceil(n/2) remain.  Round r: every k with k mod 2^(r+1) = 2^r sends to
 * k - 2^r.  A segmented message repeats the tree once per segment, a segment
 * starting only after the previous one is complete (Section IV: all processes
 * must finish before the next segment starts).                              */
int orc_binomial(int p, int q, const int64_t *sizes, int64_t A, int64_t B, int64_t G,
                 orc_event_t *events, int64_t *completion)
{
    if (p < 1 || q < 1 || !sizes) return ORC_BAD_ARG;
    int L = orc_ceil_log2(p);
    int64_t round_len = round_length(q, sizes, A, B, G);
    size_t ne = 0;
    for (int j = 0; j < q; j++) {
        for (int r = 0; r < L; r++) {
            int64_t half = (int64_t)1 << r;
            for (int64_t k = half; k < p; k += 2 * half) {
                if (events) {
                    events[ne].seg = j; events[ne].src = (int32_t)k; events[ne].dst = (int32_t)(k - half);
                    events[ne].kind = 0; events[ne].t_start = ((int64_t)j * L + r) * round_len;
                }
                ne++;
            }
        }
    }
    if (completion) *completion = (int64_t)q * L * round_len;
    return ORC_OK;
}

/* Pipeline: process k sends segment i to k-1 once k+1..p-1 are reduced for
 * it.  Unidirectional: a process alternates receive / send, so segment i
 * leaves process k in round (p-1-k) + 2i; bidirectional: (p-1-k) + i.       */
int orc_pipeline(int p, int q, const int64_t *sizes, int64_t A, int64_t B, int64_t G, int bidir,
                 orc_event_t *events, int64_t *completion)
{
    if (p < 1 || q < 1 || !sizes) return ORC_BAD_ARG;
    int64_t round_len = round_length(q, sizes, A, B, G);
    int stride = bidir ? 1 : 2;
    size_t ne = 0;
    for (int i = 0; i < q; i++) {
        for (int k = p - 1; k >= 1; k--) {
            if (events) {
                events[ne].seg = i; events[ne].src = k; events[ne].dst = k - 1; events[ne].kind = 0;
                events[ne].t_start = ((int64_t)(p - 1 - k) + (int64_t)stride * i) * round_len;
            }
            ne++;
        }
    }
    if (completion) *completion = p < 2 ? 0 : ((int64_t)(p - 1) + (int64_t)stride * (q - 1)) * round_len;
    return ORC_OK;
}

/* Binary tree in heap order (children of k: 2k+1, 2k+2), depth
 * D = ceil(log2(p+1)) - 1.  The two children of a node send in turn, left
 * first, so one step is two rounds.  A node at depth d sends segment i in
 * round 2(D-d) + [right child] + 4i (unidirectional: a node receives twice
 * and sends once per segment, its send must not meet its next receive) or
 * + 2i (bidirectional).  Leaves of an incomplete last level are the "extra"
 * processes reduced in the first step.                                       */
int orc_binary(int p, int q, const int64_t *sizes, int64_t A, int64_t B, int64_t G, int bidir,
               orc_event_t *events, int64_t *completion)
{
    if (p < 1 || q < 1 || !sizes) return ORC_BAD_ARG;
    int D = orc_ceil_log2((int64_t)p + 1) - 1;
    int64_t round_len = round_length(q, sizes, A, B, G);
    int stride = bidir ? 2 : 4;
    size_t ne = 0;
    int64_t rounds = 0;
    for (int i = 0; i < q; i++) {
        for (int k = 1; k < p; k++) {
            int d = 0;
            for (int v = k; v > 0; v = (v - 1) / 2) d++;
            int right = (k % 2 == 0);
            int64_t round = (int64_t)2 * (D - d) + right + (int64_t)stride * i;
            if (round + 1 > rounds) rounds = round + 1;
            if (events) {
                events[ne].seg = i; events[ne].src = k; events[ne].dst = (k - 1) / 2; events[ne].kind = 0;
                events[ne].t_start = round * round_len;
            }
            ne++;
        }
    }
    /* 2D + stride (q-1) rounds as soon as the root has a right child (p >= 3) */
    if (completion) *completion = rounds * round_len;
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Butterfly (Section III): reduce-scatter by recursive halving, then gather */
/* by recursive doubling, bidirectional ports, for p a power of two.  For    */
/* other p (the paper only points to an improved algorithm it does not       */
/* describe) the processes beyond the largest power of two first send their  */
/* whole message to a partner below it, which combines it; the power-of-two  */
/* algorithm then runs on the rest.  PARITY UNPINNED for that extension: the */
/* paper fixes nothing about it; only validity and the contribution          */
/* invariant are checked.  Distance                                          */
/* p/2 first; of an exchanging pair the process with the distance bit clear  */
/* keeps the lower half [lo, mid), mid = lo + floor((hi-lo)/2).  A "segment" */
/* in the event list is a final chunk c (the range process c owns after the  */
/* first phase): one combine event per (chunk, round) and receiver, then     */
/* store-only events for the gather to process 0.  Every message of a round  */
/* starts together; a round lasts as long as its largest message.            */
/* n = message length in elements, esize = size units per element.           */
/* chunk_off[p+1] receives the chunk boundaries in elements.                 */
/* Event count: P(P-1) + (P/2) log2 P + (p-P) P, P the power of two used.     */
/* ------------------------------------------------------------------------- */
int orc_butterfly(int p_all, int64_t n, int64_t esize, int64_t A, int64_t B, int64_t G,
                  orc_event_t *events, int64_t *chunk_off, int64_t *completion)
{
    if (p_all < 1 || n < 0) return ORC_BAD_ARG;
    /* p = largest power of two not above p_all; the r = p_all - p processes beyond it are folded in first */
    int p = 1;
    while (2 * p <= p_all) p *= 2;
    int r_extra = p_all - p;
    int L = orc_ceil_log2(p);
    int64_t *lo = malloc(8 * (size_t)p), *hi = malloc(8 * (size_t)p);
    int64_t *clo = malloc(8 * (size_t)p), *chi = malloc(8 * (size_t)p);
    if (!lo || !hi || !clo || !chi) { free(lo); free(hi); free(clo); free(chi); return ORC_NOMEM; }
    for (int k = 0; k < p; k++) { lo[k] = 0; hi[k] = n; }
    /* final chunk of process c = its range after all halvings */
    for (int c = 0; c < p; c++) {
        int64_t l = 0, h = n;
        for (int r = 0; r < L; r++) {
            int d = p >> (r + 1);
            int64_t mid = l + (h - l) / 2;
            if (c & d) l = mid; else h = mid;
        }
        clo[c] = l; chi[c] = h;
    }
    if (chunk_off) { for (int c = 0; c < p; c++) chunk_off[c] = clo[c]; chunk_off[p] = n; }
    size_t ne = 0;
    int64_t t = 0;
    if (r_extra > 0) {                               /* fold: process p + i sends its whole message to i */
        for (int i = 0; i < r_extra; i++) {
            for (int c = 0; c < p; c++) {
                if (events) {
                    events[ne].seg = c; events[ne].src = p + i; events[ne].dst = i;
                    events[ne].kind = 0; events[ne].t_start = 0;
                }
                ne++;
            }
        }
        t = t_comm(A, B, n * esize) + t_comp(G, n * esize);
    }
    for (int r = 0; r < L; r++) {
        int d = p >> (r + 1);
        int64_t longest = 0;
        for (int k = 0; k < p; k++) {               /* k receives from k ^ d */
            int64_t mid = lo[k] + (hi[k] - lo[k]) / 2;
            int64_t klo = (k & d) ? mid : lo[k], khi = (k & d) ? hi[k] : mid;
            int64_t bytes = (khi - klo) * esize;
            int64_t dur = t_comm(A, B, bytes) + t_comp(G, bytes);
            if (dur > longest) longest = dur;
            for (int c = 0; c < p; c++) {           /* chunks inside the kept half */
                if ((c & ~(d - 1)) != (k & ~(d - 1))) continue;
                if (events) {
                    events[ne].seg = c; events[ne].src = k ^ d; events[ne].dst = k;
                    events[ne].kind = 0; events[ne].t_start = t;
                }
                ne++;
            }
        }
        for (int k = 0; k < p; k++) {
            int64_t mid = lo[k] + (hi[k] - lo[k]) / 2;
            if (k & d) lo[k] = mid; else hi[k] = mid;
        }
        t += longest;
    }
    for (int d = 1; d < p; d *= 2) {                /* gather: k sends chunks [k, k+d) to k-d */
        int64_t longest = 0;
        for (int k = d; k < p; k += 2 * d) {
            int64_t bytes = (chi[k + d - 1] - clo[k]) * esize;
            int64_t dur = t_comm(A, B, bytes);
            if (dur > longest) longest = dur;
            for (int c = k; c < k + d; c++) {
                if (events) {
                    events[ne].seg = c; events[ne].src = k; events[ne].dst = k - d;
                    events[ne].kind = 1; events[ne].t_start = t;
                }
                ne++;
            }
        }
        t += longest;
    }
    if (completion) *completion = t;
    free(lo); free(hi); free(clo); free(chi);
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Validity of an event list under the model of Section II and Lemma 1.      */
/* Events that share (src, dst, t_start) form ONE message whose size is the  */
/* sum of their segment sizes (only the butterfly sends several chunks in    */
/* one message).  A message occupies the sender for t_comm and the receiver  */
/* for t_comm (+ t_comp when it combines).  Checks, in this order; the       */
/* return value names the first rule broken:                                 */
/*   1 malformed event (index out of range, src = dst, negative time)        */
/*   2 the root sends a combine event            (Lemma 1 (ii); tree_rules)  */
/*   3 some non-root process does not send some segment exactly once         */
/*                                               (Section IV; tree_rules)    */
/*   4 a port is used twice at once (unidirectional: a process does one      */
/*     thing at a time; bidirectional: one send and one receive), or a       */
/*     communication overlaps a computation on the same process (Section II) */
/*   5 a process sends a segment before every receive of that segment into   */
/*     it has been combined, or receives a segment it has already sent       */
/*   6 in_order: a process touches segment j after a later one (Section V)   */
/* tree_rules = 1 for everything except the butterfly.  *last_end receives    */
/* the end of the last activity (communication or computation).              */
/* ------------------------------------------------------------------------- */
typedef struct { int64_t a, b; int kind; } ivl_t;   /* kind: 0 send, 1 receive port, 2 compute */

static int cmp_ivl(const void *x, const void *y)
{
    const ivl_t *u = x, *v = y;
    if (u->a != v->a) return u->a < v->a ? -1 : 1;
    if (u->b != v->b) return u->b < v->b ? -1 : 1;
    return 0;
}

static int cmp_msg(const void *x, const void *y)
{
    const orc_event_t *u = x, *v = y;
    if (u->t_start != v->t_start) return u->t_start < v->t_start ? -1 : 1;
    if (u->src != v->src) return u->src < v->src ? -1 : 1;
    if (u->dst != v->dst) return u->dst < v->dst ? -1 : 1;
    if (u->seg != v->seg) return u->seg < v->seg ? -1 : 1;
    return 0;
}

typedef struct { int32_t dst, seg, kind; int64_t t_start, t_done; } arrival_t;

static int cmp_arrival(const void *x, const void *y)
{
    const arrival_t *u = x, *v = y;
    if (u->dst != v->dst) return u->dst < v->dst ? -1 : 1;
    if (u->seg != v->seg) return u->seg < v->seg ? -1 : 1;
    return 0;
}

int orc_validate(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *sizes,
                 int64_t A, int64_t B, int64_t G, int bidir, int tree_rules, int in_order,
                 int64_t *last_end_out)
{
    if (n_ev < 0 || p < 1 || q < 1) return 1;
    for (int64_t e = 0; e < n_ev; e++) {
        const orc_event_t *v = &ev_in[e];
        if (v->seg < 0 || v->seg >= q || v->src < 0 || v->src >= p || v->dst < 0 || v->dst >= p ||
            v->src == v->dst || v->t_start < 0 || (v->kind != 0 && v->kind != 1)) return 1;
    }
    if (tree_rules) {
        int *cnt = calloc((size_t)p * (size_t)q, sizeof(int));
        int bad = 0;
        for (int64_t e = 0; e < n_ev; e++) {
            if (ev_in[e].kind != 0) { bad = 1; break; }
            if (ev_in[e].src == 0) { bad = 2; break; }
            cnt[(size_t)ev_in[e].src * q + ev_in[e].seg]++;
        }
        if (!bad) for (int i = 1; i < p && !bad; i++) for (int j = 0; j < q; j++)
            if (cnt[(size_t)i * q + j] != 1) { bad = 3; break; }
        free(cnt);
        if (bad) return bad;
    }
    size_t cap = (size_t)(n_ev ? n_ev : 1);
    orc_event_t *ev = malloc(sizeof(orc_event_t) * cap);
    memcpy(ev, ev_in, sizeof(orc_event_t) * (size_t)n_ev);
    qsort(ev, (size_t)n_ev, sizeof(orc_event_t), cmp_msg);
    /* per event: is it the first of its message, the message's t_comm and t_comp,
     * and the instant the receiver starts combining                            */
    char *first = malloc(cap);
    int64_t *m_tc = malloc(8 * cap), *m_tp = malloc(8 * cap), *m_cs = malloc(8 * cap);
    for (int64_t e = 0; e < n_ev;) {
        int64_t f = e, bytes = 0;
        while (f < n_ev && ev[f].t_start == ev[e].t_start && ev[f].src == ev[e].src && ev[f].dst == ev[e].dst) {
            bytes += sizes[ev[f].seg]; f++;
        }
        for (int64_t g = e; g < f; g++) {
            first[g] = (g == e);
            m_tc[g] = t_comm(A, B, bytes);
            m_tp[g] = ev[g].kind == 0 ? t_comp(G, bytes) : 0;
            m_cs[g] = ev[g].t_start + m_tc[g];
        }
        e = f;
    }
    /* bidirectional ports: a process may be sending while it receives; the
     * combination cannot overlap that send (Section II), it waits for it       */
    if (bidir) {
        for (int64_t e = 0; e < n_ev; e++) {
            if (m_tp[e] == 0) continue;
            for (int64_t f = 0; f < n_ev; f++) {           /* sends of the receiver still running */
                if (!first[f] || ev[f].src != ev[e].dst) continue;
                if (ev[f].t_start > ev[e].t_start + m_tc[e]) break;
                if (ev[f].t_start <= m_cs[e] && m_cs[e] < ev[f].t_start + m_tc[f]) m_cs[e] = ev[f].t_start + m_tc[f];
            }
        }
    }
    int rc = 0;
    int64_t last_end = 0;
    /* rule 4, process by process */
    ivl_t *iv = malloc(sizeof(ivl_t) * (3 * cap + 1));
    for (int i = 0; i < p && !rc; i++) {
        int64_t ni = 0;
        for (int64_t e = 0; e < n_ev; e++) {
            if (!first[e]) continue;
            if (ev[e].src == i) { iv[ni].a = ev[e].t_start; iv[ni].b = ev[e].t_start + m_tc[e]; iv[ni].kind = 0; ni++; }
            if (ev[e].dst == i) {
                iv[ni].a = ev[e].t_start; iv[ni].b = m_cs[e] + m_tp[e]; iv[ni].kind = 1; ni++;
                if (bidir && m_tp[e] > 0) { iv[ni].a = m_cs[e]; iv[ni].b = m_cs[e] + m_tp[e]; iv[ni].kind = 2; ni++; }
            }
        }
        for (int64_t u = 0; u < ni; u++) if (iv[u].b > last_end) last_end = iv[u].b;
        qsort(iv, (size_t)ni, sizeof(ivl_t), cmp_ivl);
        for (int64_t u = 0; u < ni && !rc; u++) {
            for (int64_t v = u + 1; v < ni && iv[v].a < iv[u].b; v++) {
                if (iv[v].b <= iv[v].a || iv[u].b <= iv[u].a) continue;      /* empty interval */
                int ku = iv[u].kind, kv = iv[v].kind;
                int clash;
                if (!bidir) clash = 1;                                       /* one thing at a time */
                else clash = (ku == kv) ||                                   /* the same port twice  */
                             (ku == 0 && kv == 2) || (ku == 2 && kv == 0);   /* send during compute  */
                if (clash) { rc = 4; break; }
            }
        }
    }
    free(iv);
    /* rule 5: data safety */
    if (!rc) {
        arrival_t *ar = malloc(sizeof(arrival_t) * cap);
        for (int64_t e = 0; e < n_ev; e++) {
            ar[e].dst = ev[e].dst; ar[e].seg = ev[e].seg; ar[e].kind = ev[e].kind;
            ar[e].t_start = ev[e].t_start; ar[e].t_done = m_cs[e] + m_tp[e];
        }
        qsort(ar, (size_t)n_ev, sizeof(arrival_t), cmp_arrival);
        for (int64_t e = 0; e < n_ev && !rc; e++) {
            if (ev[e].kind != 0) continue;
            arrival_t key; key.dst = ev[e].src; key.seg = ev[e].seg;
            int64_t lo = 0, hi = n_ev;                     /* first arrival of (src, seg) */
            while (lo < hi) { int64_t mid = (lo + hi) / 2; if (cmp_arrival(&ar[mid], &key) < 0) lo = mid + 1; else hi = mid; }
            for (int64_t f = lo; f < n_ev && cmp_arrival(&ar[f], &key) == 0; f++) {
                if (ar[f].kind != 0) continue;
                if (ar[f].t_done > ev[e].t_start) { rc = 5; break; }   /* not yet combined, or arrives after */
            }
        }
        free(ar);
    }
    /* rule 6: in order */
    if (!rc && in_order) {
        int *prev_seg = malloc(sizeof(int) * (size_t)p);
        for (int i = 0; i < p; i++) prev_seg[i] = -1;
        for (int64_t e = 0; e < n_ev && !rc; e++) {        /* ev is sorted by time */
            int who[2] = { ev[e].src, ev[e].dst };
            for (int w = 0; w < 2; w++) {
                if (ev[e].seg < prev_seg[who[w]]) { rc = 6; break; }
                prev_seg[who[w]] = ev[e].seg;
            }
        }
        free(prev_seg);
    }
    if (last_end_out) *last_end_out = last_end;
    free(ev); free(first); free(m_tc); free(m_tp); free(m_cs);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* "Every process's data enters the root exactly once per segment"           */
/* (Section IV: each processor except the root must be reduced for each      */
/* segment).  Replays the events on multisets of process indices instead of  */
/* values.  Returns 0 when, for every segment, the root ends up holding each */
/* of 0..p-1 exactly once; otherwise 1 + the first offending segment.        */
/* ------------------------------------------------------------------------- */
static int cmp_time(const void *x, const void *y)
{
    const orc_event_t *u = x, *v = y;
    if (u->t_start != v->t_start) return u->t_start < v->t_start ? -1 : 1;
    if (u->dst != v->dst) return u->dst < v->dst ? -1 : 1;
    if (u->src != v->src) return u->src < v->src ? -1 : 1;
    return 0;
}

int orc_contributions(const orc_event_t *ev_in, int64_t n_ev, int p, int q)
{
    orc_event_t *ev = malloc(sizeof(orc_event_t) * (size_t)(n_ev ? n_ev : 1));
    memcpy(ev, ev_in, sizeof(orc_event_t) * (size_t)n_ev);
    qsort(ev, (size_t)n_ev, sizeof(orc_event_t), cmp_time);
    int32_t *have = malloc(sizeof(int32_t) * (size_t)p * (size_t)p);   /* have[i][k] = copies of x_k in process i */
    int rc = 0;
    for (int j = 0; j < q && !rc; j++) {
        memset(have, 0, sizeof(int32_t) * (size_t)p * (size_t)p);
        for (int i = 0; i < p; i++) have[(size_t)i * p + i] = 1;
        for (int64_t e = 0; e < n_ev; e++) {
            if (ev[e].seg != j) continue;
            int32_t *hb = have + (size_t)ev[e].dst * p, *ha = have + (size_t)ev[e].src * p;
            for (int k = 0; k < p; k++) hb[k] = (ev[e].kind == 0 ? hb[k] : 0) + ha[k];
        }
        for (int k = 0; k < p; k++) if (have[k] != 1) { rc = 1 + j; break; }
    }
    free(have); free(ev);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* O2: the reduction in schedule order.  x[i] points to process i's n        */
/* elements; segment j covers elements [seg_off[j], seg_off[j+1]).  For each */
/* segment every process starts from its own data; the events of the segment */
/* are replayed in start-time order (events that start together have         */
/* different receivers and commute), the receiver combining the segment it   */
/* holds (left operand) with the one that arrives; what process 0 holds at   */
/* the end is the result.                                                    */
/*   op 0: sum   (int32: wrap-around; fp32: one IEEE round-to-nearest add)   */
/*   op 1: max   (incoming > held ? incoming : held)                         */
/*   op 2: min   (incoming < held ? incoming : held)                         */
/*   op 3: product (int32: wrap-around; fp32: one IEEE multiply)             */
/* ------------------------------------------------------------------------- */
static uint32_t comb_i32(uint32_t held, uint32_t in, int op)
{
    if (op == 0) return held + in;
    if (op == 3) return held * in;
    if (op == 1) return ((int32_t)in > (int32_t)held) ? in : held;
    return ((int32_t)in < (int32_t)held) ? in : held;
}

static float comb_f32(float held, float in, int op)
{
    if (op == 0) return held + in;
    if (op == 3) return held * in;
    if (op == 1) return (in > held) ? in : held;
    return (in < held) ? in : held;
}

/* Threads this build runs the evaluators on (1 without OpenMP). */
int orc_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* The calling thread's share [lo, hi) of a segment's len elements (all of them without OpenMP): the
 * same share of the `longest` places of the accumulators for every segment, clipped to the segment, so
 * that a thread which is already on the next segment never touches a place another thread still uses. */
static void my_share(int64_t len, int64_t longest, int64_t *lo, int64_t *hi)
{
#ifdef _OPENMP
    const int64_t T = omp_get_num_threads(), t = omp_get_thread_num();
#else
    const int64_t T = 1, t = 0;
#endif
    *lo = longest * t / T;
    *hi = longest * (t + 1) / T;
    if (*hi > len) *hi = len;
    if (*lo > len) *lo = len;
}

static int cmp_seg_time(const void *x, const void *y)
{
    const orc_event_t *u = x, *v = y;
    if (u->seg != v->seg) return u->seg < v->seg ? -1 : 1;
    return cmp_time(x, y);
}

static orc_event_t *sorted_by_segment(const orc_event_t *ev_in, int64_t n_ev)
{
    orc_event_t *ev = malloc(sizeof(orc_event_t) * (size_t)(n_ev ? n_ev : 1));
    if (!ev) return NULL;
    memcpy(ev, ev_in, sizeof(orc_event_t) * (size_t)n_ev);
    qsort(ev, (size_t)n_ev, sizeof(orc_event_t), cmp_seg_time);
    return ev;
}

int orc_reduce_i32(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *seg_off,
                   const int32_t *const *x, int32_t *out, int op)
{
    orc_event_t *ev = sorted_by_segment(ev_in, n_ev);
    if (!ev) return ORC_NOMEM;
    int64_t longest = 0;
    for (int j = 0; j < q; j++) if (seg_off[j + 1] - seg_off[j] > longest) longest = seg_off[j + 1] - seg_off[j];
    uint32_t *acc = malloc(sizeof(uint32_t) * (size_t)p * (size_t)(longest ? longest : 1));
    if (!acc) { free(ev); return ORC_NOMEM; }
#pragma omp parallel
    {
    int64_t e = 0;
    for (int j = 0; j < q; j++) {
        int64_t len = seg_off[j + 1] - seg_off[j], lo, hi;
        my_share(len, longest, &lo, &hi);
        for (int i = 0; i < p; i++)                    /* every process starts from its own segment */
            for (int64_t k = lo; k < hi; k++) acc[(size_t)i * longest + k] = (uint32_t)x[i][seg_off[j] + k];
        for (; e < n_ev && ev[e].seg == j; e++) {
            uint32_t *held = acc + (size_t)ev[e].dst * longest, *in = acc + (size_t)ev[e].src * longest;
            if (ev[e].kind == 0) for (int64_t k = lo; k < hi; k++) held[k] = comb_i32(held[k], in[k], op);
            else for (int64_t k = lo; k < hi; k++) held[k] = in[k];
        }
        for (int64_t k = lo; k < hi; k++) out[seg_off[j] + k] = (int32_t)acc[k];
    }
    }
    free(acc); free(ev);
    return ORC_OK;
}

int orc_reduce_f32(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *seg_off,
                   const float *const *x, float *out, int op)
{
    orc_event_t *ev = sorted_by_segment(ev_in, n_ev);
    if (!ev) return ORC_NOMEM;
    int64_t longest = 0;
    for (int j = 0; j < q; j++) if (seg_off[j + 1] - seg_off[j] > longest) longest = seg_off[j + 1] - seg_off[j];
    float *acc = malloc(sizeof(float) * (size_t)p * (size_t)(longest ? longest : 1));
    if (!acc) { free(ev); return ORC_NOMEM; }
#pragma omp parallel
    {
    int64_t e = 0;
    for (int j = 0; j < q; j++) {
        int64_t len = seg_off[j + 1] - seg_off[j], lo, hi;
        my_share(len, longest, &lo, &hi);
        for (int i = 0; i < p; i++)
            for (int64_t k = lo; k < hi; k++) acc[(size_t)i * longest + k] = x[i][seg_off[j] + k];
        for (; e < n_ev && ev[e].seg == j; e++) {
            float *held = acc + (size_t)ev[e].dst * longest, *in = acc + (size_t)ev[e].src * longest;
            if (ev[e].kind == 0) for (int64_t k = lo; k < hi; k++) held[k] = comb_f32(held[k], in[k], op);
            else for (int64_t k = lo; k < hi; k++) held[k] = in[k];
        }
        for (int64_t k = lo; k < hi; k++) out[seg_off[j] + k] = acc[k];
    }
    }
    free(acc); free(ev);
    return ORC_OK;
}

/* bf16 elements combined in fp32 (the paper leaves the element type open, Fig. 2
 * caption; this is the usual meaning of "16-bit storage, 32-bit accumulation"):
 * every input is widened exactly (a bf16 is the upper half of an fp32), the
 * replay above runs on fp32 values, one IEEE fp32 operation per combine, and only
 * what process 0 holds at the end is rounded to bf16, once, to nearest with
 * ties to even.  NaN inputs are outside the parity tests.  seg_off counts
 * elements.                                                                   */
static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

static uint16_t f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);   /* NaN stays NaN */
    /* the 16 bits that are dropped: above half -> up, below -> down, exactly half -> to the even neighbour */
    uint32_t lower = u & 0xFFFFu, keep = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (keep & 1u))) keep++;
    return (uint16_t)keep;
}

/* fp16 (IEEE binary16) elements, treated the same way: widened exactly, combined in fp32, rounded once at
 * the root to nearest with ties to even (overflow goes to infinity, small results become subnormal).  The
 * conversions are the compiler's own for _Float16, which are the IEEE ones.                              */
static float f16_to_f32(uint16_t h)
{
    _Float16 x;
    memcpy(&x, &h, sizeof x);
    return (float)x;
}

static uint16_t f32_to_f16(float f)
{
    _Float16 x = (_Float16)f;
    uint16_t h;
    memcpy(&h, &x, sizeof h);
    return h;
}

static int reduce_half(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *seg_off,
                       const uint16_t *const *x, uint16_t *out, int op,
                       float (*widen)(uint16_t), uint16_t (*narrow)(float))
{
    orc_event_t *ev = sorted_by_segment(ev_in, n_ev);
    if (!ev) return ORC_NOMEM;
    int64_t longest = 0;
    for (int j = 0; j < q; j++) if (seg_off[j + 1] - seg_off[j] > longest) longest = seg_off[j + 1] - seg_off[j];
    float *acc = malloc(sizeof(float) * (size_t)p * (size_t)(longest ? longest : 1));
    if (!acc) { free(ev); return ORC_NOMEM; }
    int64_t e = 0;
    for (int j = 0; j < q; j++) {
        int64_t len = seg_off[j + 1] - seg_off[j];
        for (int i = 0; i < p; i++)
            for (int64_t k = 0; k < len; k++) acc[(size_t)i * longest + k] = widen(x[i][seg_off[j] + k]);
        for (; e < n_ev && ev[e].seg == j; e++) {
            float *held = acc + (size_t)ev[e].dst * longest, *in = acc + (size_t)ev[e].src * longest;
            if (ev[e].kind == 0) for (int64_t k = 0; k < len; k++) held[k] = comb_f32(held[k], in[k], op);
            else for (int64_t k = 0; k < len; k++) held[k] = in[k];
        }
        for (int64_t k = 0; k < len; k++) out[seg_off[j] + k] = narrow(acc[k]);
    }
    free(acc); free(ev);
    return ORC_OK;
}

int orc_reduce_bf16(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *seg_off,
                    const uint16_t *const *x, uint16_t *out, int op)
{
    return reduce_half(ev_in, n_ev, p, q, seg_off, x, out, op, bf16_to_f32, f32_to_bf16);
}

int orc_reduce_f16(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *seg_off,
                   const uint16_t *const *x, uint16_t *out, int op)
{
    return reduce_half(ev_in, n_ev, p, q, seg_off, x, out, op, f16_to_f32, f32_to_f16);
}

/* The same for the 8-byte element types: int64 wraps modulo 2^64, fp64 is one
 * IEEE round-to-nearest operation per combine.  seg_off counts elements.     */
static uint64_t comb_i64(uint64_t held, uint64_t in, int op)
{
    if (op == 0) return held + in;
    if (op == 3) return held * in;
    if (op == 1) return ((int64_t)in > (int64_t)held) ? in : held;
    return ((int64_t)in < (int64_t)held) ? in : held;
}

static double comb_f64(double held, double in, int op)
{
    if (op == 0) return held + in;
    if (op == 3) return held * in;
    if (op == 1) return (in > held) ? in : held;
    return (in < held) ? in : held;
}

int orc_reduce_i64(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *seg_off,
                   const int64_t *const *x, int64_t *out, int op)
{
    orc_event_t *ev = sorted_by_segment(ev_in, n_ev);
    if (!ev) return ORC_NOMEM;
    int64_t longest = 0;
    for (int j = 0; j < q; j++) if (seg_off[j + 1] - seg_off[j] > longest) longest = seg_off[j + 1] - seg_off[j];
    uint64_t *acc = malloc(sizeof(uint64_t) * (size_t)p * (size_t)(longest ? longest : 1));
    if (!acc) { free(ev); return ORC_NOMEM; }
    int64_t e = 0;
    for (int j = 0; j < q; j++) {
        int64_t len = seg_off[j + 1] - seg_off[j];
        for (int i = 0; i < p; i++)
            for (int64_t k = 0; k < len; k++) acc[(size_t)i * longest + k] = (uint64_t)x[i][seg_off[j] + k];
        for (; e < n_ev && ev[e].seg == j; e++) {
            uint64_t *held = acc + (size_t)ev[e].dst * longest, *in = acc + (size_t)ev[e].src * longest;
            if (ev[e].kind == 0) for (int64_t k = 0; k < len; k++) held[k] = comb_i64(held[k], in[k], op);
            else for (int64_t k = 0; k < len; k++) held[k] = in[k];
        }
        for (int64_t k = 0; k < len; k++) out[seg_off[j] + k] = (int64_t)acc[k];
    }
    free(acc); free(ev);
    return ORC_OK;
}

int orc_reduce_f64(const orc_event_t *ev_in, int64_t n_ev, int p, int q, const int64_t *seg_off,
                   const double *const *x, double *out, int op)
{
    orc_event_t *ev = sorted_by_segment(ev_in, n_ev);
    if (!ev) return ORC_NOMEM;
    int64_t longest = 0;
    for (int j = 0; j < q; j++) if (seg_off[j + 1] - seg_off[j] > longest) longest = seg_off[j + 1] - seg_off[j];
    double *acc = malloc(sizeof(double) * (size_t)p * (size_t)(longest ? longest : 1));
    if (!acc) { free(ev); return ORC_NOMEM; }
    int64_t e = 0;
    for (int j = 0; j < q; j++) {
        int64_t len = seg_off[j + 1] - seg_off[j];
        for (int i = 0; i < p; i++)
            for (int64_t k = 0; k < len; k++) acc[(size_t)i * longest + k] = x[i][seg_off[j] + k];
        for (; e < n_ev && ev[e].seg == j; e++) {
            double *held = acc + (size_t)ev[e].dst * longest, *in = acc + (size_t)ev[e].src * longest;
            if (ev[e].kind == 0) for (int64_t k = 0; k < len; k++) held[k] = comb_f64(held[k], in[k], op);
            else for (int64_t k = 0; k < len; k++) held[k] = in[k];
        }
        for (int64_t k = 0; k < len; k++) out[seg_off[j] + k] = acc[k];
    }
    free(acc); free(ev);
    return ORC_OK;
}

/* Order-free fp64 reference: sum_i (double)x_i[e], and sum_i |x_i[e]| for the
 * error bound; for max the exact maximum as a double.                        */
int orc_reference_f64(int p, int64_t n, const float *const *x, double *ref, double *abs_sum, int op)
{
    for (int64_t e = 0; e < n; e++) {
        double s = (op == 0) ? 0.0 : (double)x[0][e], a = 0.0;
        for (int i = 0; i < p; i++) {
            double v = (double)x[i][e];
            if (op == 0) s += v; else if (v > s) s = v;
            a += v < 0 ? -v : v;
        }
        ref[e] = s;
        if (abs_sum) abs_sum[e] = a;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Section VIII: a message of 10 units, every one of its 512 segmentations   */
/* (compositions of 10).  Bit k (0..8) of the index set = a cut after unit   */
/* k+1.  times[512] receives the uni-greedy completion time of each with     */
/* beta = 1.                                                                 */
/* ------------------------------------------------------------------------- */
int orc_unequal_times(int p, int64_t A, int64_t G, int64_t *times)
{
    for (int mask = 0; mask < 512; mask++) {
        int64_t sizes[10];
        int q = 0;
        int64_t run = 0;
        for (int u = 0; u < 10; u++) {
            run++;
            if (u == 9 || (mask >> u) & 1) { sizes[q++] = run; run = 0; }
        }
        int rc = orc_uni_greedy(p, q, sizes, A, 1, G, NULL, &times[mask]);
        if (rc) return rc;
    }
    return ORC_OK;
}
