/*
 * bcast_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-threaded CPU statement of the round-optimal broadcast
 * schedule of Traff, "Optimal Broadcast Schedules in Logarithmic Time ..."
 * (arXiv 2407.18004).  It exists only so that the CUDA library can be compared
 * with something written straight from the paper.  It shares no code, header,
 * table or helper with the CUDA path and must never be linked into, imported
 * by or called from it.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg use it.
 *
 * The receive schedule has no closed definition: it is whatever Algorithm 5
 * (with Algorithms 2, 3 and 4) produces, so those are executed here step by
 * step, with the paper's variable names, a real doubly linked list and real
 * recursion.  The send schedule HAS a plain definition (Section 2.3:
 * sendblock[k] of r is recvblock[k] of (r+skip[k]) mod p) and that definition
 * is what the table functions use.  Algorithm 6 is kept as a second,
 * independent routine (oracle_sendschedule_alg6) that the tests cross-check
 * against the definition.
 *
 * Readings taken where the paper is silent (all listed in the design notes):
 *  - Algorithm 4: r, r', s, e are passed by value; k is passed by value and
 *    handed back as the return value; recvblock/next/prev are shared.
 *  - Algorithm 4's recursive call passes the same e, so the callee tests it
 *    once more.  Kept as printed.
 *  - skip[k+1] is never needed with k = q; the oracle records it in `oob`
 *    if that ever happens instead of reading past the array.
 *  - p = 1 gives q = 0 and empty schedules; Algorithm 3's repeat-loop is not
 *    entered then.
 *  - all quantities are 64-bit: p+r, 2p and r'+skip[e] exceed 32 bits for
 *    large p.
 *
 * Every function is pinned by the CPU tests against values the paper prints
 * (Tables 1-3, the p=11 baseblock string), closed forms (powers of two), the
 * four correctness conditions, the doubling observations and a brute-force
 * broadcast simulation.  No function here is "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAXQ 64

typedef struct {
    int      q;
    int64_t  p;
    int64_t  skip[ORACLE_MAXQ + 2];
    /* linked list over indices -1..q, stored with an offset of one */
    int      next_[ORACLE_MAXQ + 3];
    int      prev_[ORACLE_MAXQ + 3];
    int      recvblock[ORACLE_MAXQ + 1];
    /* instrumentation for the bounds the paper states (Lemmas 5 and 6) */
    int64_t  calls;      /* recursive calls, the first invocation not counted */
    int64_t  iters;      /* while-loop iterations over all calls              */
    int64_t  retests;    /* iterations that are a callee's first look at the
                            very index its caller just tested                 */
    int64_t  retest_hits;/* how many of those passed the outer test           */
    int64_t  oob;        /* skip[k+1] wanted with k >= q                      */
    int64_t  rprime[ORACLE_MAXQ + 1];  /* the processor r'_k accepted for round k (Lemma 4) */
} oracle_ctx;

#define NEXT(c, e) ((c)->next_[(e) + 1])
#define PREV(c, e) ((c)->prev_[(e) + 1])

/* q = ceil(log2 p)  (Section 2, "we let p denote ... and take q = ...") */
int oracle_q(int64_t p)
{
    int q = 0;
    if (p < 1) return -1;
    while (((int64_t)1 << q) < p) q++;
    return q;
}

/* Algorithm 2: skips by repeated halving with rounding up. skip has q+1 slots. */
int oracle_skips(int64_t p, int64_t *skip)
{
    int q = oracle_q(p);
    int k;
    if (q < 0) return -1;
    k = q;
    skip[k] = p;
    while (k > 0) {
        skip[k - 1] = skip[k] - skip[k] / 2;
        k = k - 1;
    }
    return q;
}

/* Algorithm 3: smallest index of the canonical skip sequence of r; q for r=0. */
static int baseblock_(const oracle_ctx *c, int64_t r)
{
    int k = c->q;
    int64_t rp = 0;
    if (c->q == 0) return c->q;
    do {
        k = k - 1;
        if (rp + c->skip[k] == r) return k;
        else if (rp + c->skip[k] < r) rp = rp + c->skip[k];
    } while (k != 0);
    return c->q;
}

/* Algorithm 4: greedy depth-first search with removal of accepted indices. */
static int allblocks_(oracle_ctx *c, int64_t r, int64_t rp, int64_t s, int e, int k,
                      int fresh_call)
{
    const int64_t *skip = c->skip;
    int first = fresh_call;
    while (e != -1) {
        c->iters++;
        if (first) c->retests++;
        if (rp + skip[e] <= r - skip[k] && rp + skip[e] < s) {
            if (first) c->retest_hits++;
            if (k >= c->q) { c->oob++; return k; }
            if (rp + skip[e] <= r - skip[k + 1]) {
                c->calls++;
                k = allblocks_(c, r, rp + skip[e], s, e, k, 1);
            }
            if (k >= c->q) { c->oob++; return k; }
            if (rp > r - skip[k + 1]) return k;
            s = rp + skip[e];
            c->rprime[k] = s;
            c->recvblock[k] = e;
            k = k + 1;
            NEXT(c, PREV(c, e)) = NEXT(c, e);
            PREV(c, NEXT(c, e)) = PREV(c, e);
        }
        first = 0;
        e = NEXT(c, e);
    }
    return k;
}

static int ctx_init_(oracle_ctx *c, int64_t p)
{
    memset(c, 0, sizeof(*c));
    c->p = p;
    c->q = oracle_skips(p, c->skip);
    if (c->q < 0 || c->q > ORACLE_MAXQ) return -1;
    return 0;
}

/* Algorithm 5: receive schedule of virtual rank r (root is rank 0). */
static int recvschedule_(oracle_ctx *c, int64_t r, int *recvblock, int *b_out)
{
    int q = c->q, e, k, b;
    for (e = 0; e <= q; e++) { NEXT(c, e) = e - 1; PREV(c, e) = e + 1; }
    PREV(c, q) = -1; NEXT(c, -1) = q; PREV(c, -1) = 0;
    b = baseblock_(c, r);
    NEXT(c, PREV(c, b)) = NEXT(c, b);
    PREV(c, NEXT(c, b)) = PREV(c, b);
    k = allblocks_(c, c->p + r, 0, c->p + c->p, q, 0, 0);
    for (k = 0; k < q; k++) {
        if (c->recvblock[k] == q) recvblock[k] = b;
        else recvblock[k] = c->recvblock[k] - q;
    }
    if (b_out) *b_out = b;
    return 0;
}

int oracle_baseblock(int64_t p, int64_t r)
{
    oracle_ctx c;
    if (ctx_init_(&c, p) || r < 0 || r >= p) return -1;
    return baseblock_(&c, r);
}

/*
 * Receive schedule of virtual rank r.  stats (may be NULL) receives
 * {recursive calls, while iterations, re-test iterations, re-test hits, oob}.
 */
int oracle_recvschedule(int64_t p, int64_t r, int32_t *recvblock, int64_t *stats)
{
    oracle_ctx c;
    int tmp[ORACLE_MAXQ + 1], k;
    if (ctx_init_(&c, p) || r < 0 || r >= p) return -1;
    /* poison so that an entry the search never wrote is seen by the tests */
    for (k = 0; k <= c.q; k++) c.recvblock[k] = -1000;
    recvschedule_(&c, r, tmp, NULL);
    for (k = 0; k < c.q; k++) recvblock[k] = tmp[k];
    if (stats) {
        stats[0] = c.calls; stats[1] = c.iters; stats[2] = c.retests;
        stats[3] = c.retest_hits; stats[4] = c.oob;
    }
    return c.q;
}

/*
 * The intermediate processors r'_k (in [p, 2p), the search runs on p + r) whose
 * baseblocks make up the receive schedule of r: Lemma 4 places them in
 * [p + r - skip[k+1], p + r - skip[k]].
 */
int oracle_recv_positions(int64_t p, int64_t r, int64_t *rprime)
{
    oracle_ctx c;
    int tmp[ORACLE_MAXQ + 1], k;
    if (ctx_init_(&c, p) || r < 0 || r >= p) return -1;
    recvschedule_(&c, r, tmp, NULL);
    for (k = 0; k < c.q; k++) rprime[k] = c.rprime[k];
    return c.q;
}

/* Send schedule by its definition: q receive schedules, one entry of each. */
int oracle_sendschedule_def(int64_t p, int64_t r, int32_t *sendblock)
{
    oracle_ctx c;
    int tmp[ORACLE_MAXQ + 1], k;
    if (ctx_init_(&c, p) || r < 0 || r >= p) return -1;
    for (k = 0; k < c.q; k++) {
        int64_t t = (r + c.skip[k]) % p;
        recvschedule_(&c, t, tmp, NULL);
        sendblock[k] = tmp[k];
    }
    return c.q;
}

/*
 * Algorithm 6, as a second routine that the tests compare with the definition.
 * violations (may be NULL) receives the number of rounds that fell back to a
 * receive-schedule computation; viol_mask (may be NULL) one bit per such round.
 */
int oracle_sendschedule_alg6(int64_t p, int64_t r, int32_t *sendblock,
                             int32_t *violations, uint64_t *viol_mask)
{
    oracle_ctx c;
    int q, k, b, nviol = 0;
    int block[ORACLE_MAXQ + 1];
    uint64_t vm = 0;
    if (ctx_init_(&c, p) || r < 0 || r >= p) return -1;
    q = c.q;
    if (r == 0) {
        for (k = 0; k < q; k++) sendblock[k] = k;
    } else {
        int64_t rp, e;
        int cc;
        b = baseblock_(&c, r);
        rp = r; cc = b; e = p;
        for (k = q - 1; k >= 1; k--) {
            if (rp < c.skip[k]) {                       /* lower part */
                if (rp + c.skip[k] < e || e < c.skip[k - 1] || (k == 1 && b > 0)) {
                    sendblock[k] = cc;
                } else {                                /* violation */
                    recvschedule_(&c, (r + c.skip[k]) % p, block, NULL);
                    sendblock[k] = block[k];
                    nviol++; vm |= (uint64_t)1 << k;
                }
                if (e > c.skip[k]) e = c.skip[k];
            } else {                                    /* upper part */
                cc = k - q;
                if (k == 1 || rp > c.skip[k] || e - c.skip[k] < c.skip[k - 1]) {
                    sendblock[k] = cc;
                } else if (rp + c.skip[k] > e) {        /* violation */
                    recvschedule_(&c, (r + c.skip[k]) % p, block, NULL);
                    sendblock[k] = block[k];
                    nviol++; vm |= (uint64_t)1 << k;
                } else {
                    sendblock[k] = cc;
                }
                rp = rp - c.skip[k];
                e = e - c.skip[k];
            }
        }
        if (q > 0) sendblock[0] = b - q;
    }
    if (violations) *violations = nviol;
    if (viol_mask) *viol_mask = vm;
    return q;
}

/*
 * Tables for actual ranks a in [rank_begin, rank_end) with the given root:
 * row a-rank_begin holds the schedule of virtual rank (a-root+p) mod p
 * (Section 2: a root other than 0 is handled by renumbering).  Either output
 * may be NULL.  Row-major, q entries per row, no padding.
 *
 * Send rows follow the definition.  When the whole range [0,p) is asked for,
 * the needed receive entries are already in this call's own receive table and
 * are gathered from it; otherwise they are computed one receive schedule per
 * entry.  The two routes are compared by the tests.
 */
int oracle_schedule_table(int64_t p, int64_t root, int64_t rank_begin, int64_t rank_end,
                          int32_t *recv_out, int32_t *send_out)
{
    oracle_ctx c;
    int tmp[ORACLE_MAXQ + 1], k, q;
    int64_t a;
    int32_t *recv_tab = recv_out;
    int own = 0;
    if (ctx_init_(&c, p)) return -1;
    if (root < 0 || root >= p || rank_begin < 0 || rank_end > p || rank_begin > rank_end) return -1;
    q = c.q;
    if (q == 0) return 0;
    {
        int full = (rank_begin == 0 && rank_end == p);
        if (full && send_out && !recv_tab) {
            recv_tab = (int32_t *)malloc((size_t)p * q * sizeof(int32_t));
            if (!recv_tab) return -2;
            own = 1;
        }
        if (recv_tab) {
            for (a = rank_begin; a < rank_end; a++) {
                int64_t r = (a - root + p) % p;
                recvschedule_(&c, r, tmp, NULL);
                for (k = 0; k < q; k++) recv_tab[(a - rank_begin) * q + k] = tmp[k];
            }
        }
        if (send_out) {
            for (a = rank_begin; a < rank_end; a++) {
                for (k = 0; k < q; k++) {
                    if (full) {
                        int64_t t = (a + c.skip[k]) % p;     /* actual to-processor */
                        send_out[a * q + k] = recv_tab[t * q + k];
                    } else {
                        int64_t r = (a - root + p) % p;
                        recvschedule_(&c, (r + c.skip[k]) % p, tmp, NULL);
                        send_out[(a - rank_begin) * q + k] = tmp[k];
                    }
                }
            }
        }
    }
    if (own) free(recv_tab);
    return q;
}

/*
 * Algorithm 7 (Appendix A), the schedule part, for processor r: with every
 * processor j as root, recvblocks[j] = recvschedule((r - j + p) mod p), and then
 * sendblocks[j][k] = recvblocks[(j - skip[k] + p) mod p][k].  Rows for the roots
 * j in [root_begin, root_end); row-major, q entries per row.  When the whole
 * range [0, p) is asked for the second loop reads this call's own recvblocks,
 * as printed; for a window the needed rows of other roots are computed one
 * receive schedule per entry.
 */
int oracle_allbroadcast_schedule(int64_t p, int64_t r, int64_t root_begin, int64_t root_end,
                                 int32_t *recvblocks, int32_t *sendblocks)
{
    oracle_ctx c;
    int tmp[ORACLE_MAXQ + 1], k, q;
    int64_t j;
    if (ctx_init_(&c, p)) return -1;
    if (r < 0 || r >= p || root_begin < 0 || root_end > p || root_begin > root_end) return -1;
    q = c.q;
    if (q == 0) return 0;
    for (j = root_begin; j < root_end; j++) {
        int64_t rp = (r - j + p) % p;
        recvschedule_(&c, rp, tmp, NULL);
        for (k = 0; k < q; k++) recvblocks[(j - root_begin) * q + k] = tmp[k];
    }
    for (j = root_begin; j < root_end; j++) {
        for (k = 0; k < q; k++) {
            int64_t f = (j - c.skip[k] + p) % p;
            if (root_begin == 0 && root_end == p) {
                sendblocks[j * q + k] = recvblocks[f * q + k];
            } else {
                recvschedule_(&c, (r - f + p) % p, tmp, NULL);
                sendblocks[(j - root_begin) * q + k] = tmp[k];
            }
        }
    }
    return q;
}

/*
 * Algorithm 1, the part that turns a schedule row into the block of one round.
 * n blocks, communication round j in [0, n-1+q): x = (q - (n-1) mod q) mod q
 * virtual rounds precede it, so i = x + j, k = i mod q, and after the shift by
 * -x (+q for i<x) and one +q per earlier use the entry reads
 * sched[k] + q*floor(i/q) - x  (Theorem 1).  Negative: nothing is transferred
 * (returns -1); above n-1: block n-1.
 */
int oracle_round_k(int q, int64_t n, int64_t j)
{
    int64_t x;
    if (q < 1 || n < 1 || j < 0 || j >= n - 1 + q) return -1;
    x = (q - (n - 1) % q) % q;
    return (int)((x + j) % q);
}

int64_t oracle_round_block(int q, int64_t n, int64_t j, const int32_t *sched_row)
{
    int64_t x, i, raw;
    int k;
    if (q < 1 || n < 1 || j < 0 || j >= n - 1 + q) return -2;
    x = (q - (n - 1) % q) % q;
    i = x + j;
    k = (int)(i % q);
    /* the printed form: subtract x, add q when k < x, then q per earlier use */
    raw = (int64_t)sched_row[k] - x;
    if (k < x) raw += q;
    {
        /* uses of entry k before round i: rounds i' in [x, i) with i' mod q = k */
        int64_t first = (k >= x) ? k : k + q;   /* first round >= x with residue k */
        int64_t uses = (i - first) / q;
        raw += uses * q;
    }
    if (raw < 0) return -1;
    if (raw > n - 1) return n - 1;
    return raw;
}

/*
 * Algorithm 1 executed as printed, for one processor: shift both schedule rows
 * by -x (+q for entries i < x), then walk rounds i = x .. n+q-1+x-1, reading
 * entry k = i mod q and adding q to it after each use.  Outputs one value per
 * communication round j = i - x: the round index k and the raw (uncapped,
 * possibly negative) receive and send block numbers.  The caller applies the
 * rules the paper leaves to the Send||Recv operation.
 */
int oracle_broadcast_rounds(int q, int64_t n, const int32_t *recvrow, const int32_t *sendrow,
                            int32_t *k_out, int64_t *recv_raw, int64_t *send_raw)
{
    int64_t rb[ORACLE_MAXQ + 1], sb[ORACLE_MAXQ + 1];
    int64_t x, i;
    int k;
    if (q < 1 || q > ORACLE_MAXQ || n < 1) return -1;
    x = (q - (n - 1) % q) % q;
    for (i = 0; i < q; i++) {
        rb[i] = (int64_t)recvrow[i] - x;
        sb[i] = (int64_t)sendrow[i] - x;
        if (i < x) { rb[i] += q; sb[i] += q; }
    }
    for (i = x; i < n + q - 1 + x; i++) {
        k = (int)(i % q);
        k_out[i - x] = k;
        recv_raw[i - x] = rb[k];
        send_raw[i - x] = sb[k];
        sb[k] += q;
        rb[k] += q;
    }
    return (int)x;
}

/*
 * Checksum of the whole schedule of p (root 0), used by the verification sweep:
 * the wrapping 64-bit sum over all ranks r and rounds k of mix(key), with
 *   key = r * 2^32 + k * 2^16 + (recv mod 256) * 2^8 + (send mod 256)
 * and mix the finaliser of the SplitMix64 generator (Steele, Lea, Flood 2014):
 *   z ^= z >> 30; z *= 0xbf58476d1ce4e5b9; z ^= z >> 27;
 *   z *= 0x94d049bb133111eb; z ^= z >> 31.
 * A sum, so that the order of evaluation does not matter.
 */
static uint64_t mix64_(uint64_t z)
{
    z ^= z >> 30; z *= 0xbf58476d1ce4e5b9ULL;
    z ^= z >> 27; z *= 0x94d049bb133111ebULL;
    z ^= z >> 31;
    return z;
}

int oracle_checksum(int64_t p, uint64_t *checksum)
{
    int q = oracle_q(p);
    int32_t *recv, *send;
    int64_t r;
    int k;
    uint64_t sum = 0;
    if (q < 0) return -1;
    if (q == 0) { *checksum = 0; return 0; }
    recv = (int32_t *)malloc((size_t)p * q * sizeof(int32_t));
    send = (int32_t *)malloc((size_t)p * q * sizeof(int32_t));
    if (!recv || !send) { free(recv); free(send); return -2; }
    oracle_schedule_table(p, 0, 0, p, recv, send);
    for (r = 0; r < p; r++)
        for (k = 0; k < q; k++) {
            uint64_t key = ((uint64_t)r << 32) | ((uint64_t)k << 16)
                         | ((uint64_t)(recv[r * q + k] & 0xff) << 8)
                         | (uint64_t)(send[r * q + k] & 0xff);
            sum += mix64_(key);
        }
    free(recv); free(send);
    *checksum = sum;
    return q;
}

/*
 * Independent (p, rank, root) queries: row i of each output has row_stride
 * entries; the first q_i hold the schedule of virtual rank
 * (rank_i - root_i + p_i) mod p_i, the rest hold `pad`.
 */
int oracle_schedule_batch(const int32_t *p, const int32_t *rank, const int32_t *root,
                          int64_t nq, int32_t row_stride, int32_t pad,
                          int32_t *recv_out, int32_t *send_out)
{
    int64_t i;
    int k;
    for (i = 0; i < nq; i++) {
        int64_t pi = p[i], r;
        int q = oracle_q(pi);
        if (q < 0 || q > row_stride || rank[i] < 0 || rank[i] >= pi || root[i] < 0 || root[i] >= pi)
            return -1;
        r = ((int64_t)rank[i] - root[i] + pi) % pi;
        if (recv_out) {
            oracle_recvschedule(pi, r, recv_out + i * row_stride, NULL);
            for (k = q; k < row_stride; k++) recv_out[i * row_stride + k] = pad;
        }
        if (send_out) {
            oracle_sendschedule_def(pi, r, send_out + i * row_stride);
            for (k = q; k < row_stride; k++) send_out[i * row_stride + k] = pad;
        }
    }
    return 0;
}

/*
 * Send rows of independent queries by Algorithm 6 (the second routine, see
 * oracle_sendschedule_alg6), padded like oracle_schedule_batch.  The tests use
 * it where q receive schedules per query (the definition) would take too long.
 */
int oracle_sendschedule_alg6_batch(const int32_t *p, const int32_t *rank, const int32_t *root,
                                   int64_t nq, int32_t row_stride, int32_t pad, int32_t *send_out)
{
    int64_t i;
    int k;
    for (i = 0; i < nq; i++) {
        int64_t pi = p[i], r;
        int q = oracle_q(pi);
        if (q < 0 || q > row_stride || rank[i] < 0 || rank[i] >= pi || root[i] < 0 || root[i] >= pi)
            return -1;
        r = ((int64_t)rank[i] - root[i] + pi) % pi;
        if (oracle_sendschedule_alg6(pi, r, send_out + i * row_stride, NULL, NULL) < 0) return -1;
        for (k = q; k < row_stride; k++) send_out[i * row_stride + k] = pad;
    }
    return 0;
}

/*
 * Algorithm 1's preamble for a whole table: the rows Broadcast() starts its
 * communication loop with when n blocks are broadcast.  With
 * x = (q - (n-1) mod q) mod q every entry has x subtracted, and the entries of
 * the rounds i < x, which are virtual and already "done", have q added.
 * In place on `rows` rows of q entries.
 */
int oracle_shift_rows(int q, int64_t n, int64_t rows, int32_t *tab)
{
    int64_t x, a;
    int i;
    if (q < 1 || n < 1 || rows < 0) return -1;
    x = (q - (n - 1) % q) % q;
    for (a = 0; a < rows; a++)
        for (i = 0; i < q; i++) {
            tab[a * q + i] = (int32_t)(tab[a * q + i] - x);
            if (i < x) tab[a * q + i] += q;
        }
    return (int)x;
}

/*
 * Algorithm 1 run by all p processors in lock-step on given schedule tables
 * (rows indexed by actual rank, as oracle_schedule_table writes them), blocks
 * moved by the rules the paper leaves to the Send||Recv operation: a negative
 * block is neither sent nor received, a block above n-1 stands for n-1,
 * nothing is sent to the root and the root receives nothing.
 *
 * Every processor keeps its own shifted copy of both rows (the preamble above)
 * and adds q to an entry after each use, as printed.  A round has two halves:
 * first every processor decides, from what it held BEFORE the round, what it
 * puts on the wire; then every processor takes what its from-processor sent.
 *
 * arrival[b * p + a]: the communication round (counted from 1) in which
 * processor a received block b; 0 for the root (it has the blocks from the
 * start); -1 if it never arrived.  A block is delivered only if the sender
 * sends exactly the block the receiver expects and held it before the round
 * and the receiver does not hold it yet.
 * stats[0] receiver expects a block, sender sends another one or nothing
 * stats[1] matching block, but the sender did not hold it before the round
 * stats[2] matching block that the receiver already holds
 * stats[3] a block is sent to a processor (not the root) that expects nothing
 * stats[4] (processor, block) pairs still missing after the last round
 * stats[5] table entries outside [-q, q-1] (they count as "nothing" in every round)
 * stats[6] blocks delivered
 * stats[7] last round in which something was delivered
 */
int oracle_simulate_broadcast(int64_t p, int64_t root, int64_t n,
                              const int32_t *recv_tab, const int32_t *send_tab,
                              int32_t *arrival, uint64_t *stats)
{
    int q = oracle_q(p);
    int64_t skip[ORACLE_MAXQ + 2];
    int64_t x, i, a, b, rounds;
    int64_t *rb, *sb, *wire;
    unsigned char *rvalid, *svalid, *wire_held;
    int k;
    if (q < 0 || n < 1 || root < 0 || root >= p) return -1;
    memset(stats, 0, 8 * sizeof(uint64_t));
    for (b = 0; b < n; b++)
        for (a = 0; a < p; a++) arrival[b * p + a] = (a == root) ? 0 : -1;
    if (q == 0) return 0;
    oracle_skips(p, skip);
    rounds = n - 1 + q;
    x = (q - (n - 1) % q) % q;
    rb = (int64_t *)malloc((size_t)p * q * sizeof(int64_t));
    sb = (int64_t *)malloc((size_t)p * q * sizeof(int64_t));
    rvalid = (unsigned char *)malloc((size_t)p * q);
    svalid = (unsigned char *)malloc((size_t)p * q);
    wire = (int64_t *)malloc((size_t)p * sizeof(int64_t));
    wire_held = (unsigned char *)malloc((size_t)p);
    if (!rb || !sb || !rvalid || !svalid || !wire || !wire_held) {
        free(rb); free(sb); free(rvalid); free(svalid); free(wire); free(wire_held);
        return -2;
    }
    for (a = 0; a < p; a++)
        for (i = 0; i < q; i++) {
            int32_t rv = recv_tab[a * q + i], sv = send_tab[a * q + i];
            rvalid[a * q + i] = (rv >= -q && rv <= q - 1);
            svalid[a * q + i] = (sv >= -q && sv <= q - 1);
            if (!rvalid[a * q + i]) stats[5]++;
            if (!svalid[a * q + i]) stats[5]++;
            rb[a * q + i] = (int64_t)rv - x;
            sb[a * q + i] = (int64_t)sv - x;
            if (i < x) { rb[a * q + i] += q; sb[a * q + i] += q; }
        }
    for (i = x; i < n + q - 1 + x; i++) {
        int64_t round = i - x + 1;                 /* communication rounds counted from 1 */
        k = (int)(i % q);
        /* first half: what goes on the wire, from the state before the round */
        for (a = 0; a < p; a++) {
            int64_t t = (a + skip[k]) % p;
            int64_t blk = sb[a * q + k];
            wire[a] = -1;
            wire_held[a] = 0;
            if (svalid[a * q + k] && blk >= 0 && t != root) {
                if (blk > n - 1) blk = n - 1;
                wire[a] = blk;
                wire_held[a] = (arrival[blk * p + a] >= 0);
            }
        }
        /* second half: every processor but the root takes what its from-processor sent */
        for (a = 0; a < p; a++) {
            int64_t f = (a - skip[k] + p) % p;
            int64_t want = rb[a * q + k];
            if (a == root) continue;
            if (!rvalid[a * q + k] || want < 0) want = -1;
            else if (want > n - 1) want = n - 1;
            if (want < 0) {
                if (wire[f] >= 0) stats[3]++;
            } else if (wire[f] != want) {
                stats[0]++;
            } else if (!wire_held[f]) {
                stats[1]++;
            } else if (arrival[want * p + a] >= 0) {
                stats[2]++;
            } else {
                arrival[want * p + a] = (int32_t)round;
                stats[6]++;
                stats[7] = (uint64_t)round;
            }
        }
        for (a = 0; a < p; a++) { sb[a * q + k] += q; rb[a * q + k] += q; }
    }
    (void)rounds;
    for (b = 0; b < n; b++)
        for (a = 0; a < p; a++)
            if (arrival[b * p + a] < 0) stats[4]++;
    free(rb); free(sb); free(rvalid); free(svalid); free(wire); free(wire_held);
    return q;
}

/*
 * The reduction of Observation 1 (item 3): Algorithm 1 with every communication
 * reversed, rounds taken downwards from (n-1+q+x)-1 to x, and the received
 * block combined into the processor's own partial result.  In the round that
 * was broadcast round i, processor a sends its partial result of block
 * recvblock[k] to its from-processor f and receives, from its to-processor t,
 * a partial result of block sendblock[k], which it adds to its own.  The same
 * exceptions, reversed: a negative block moves nothing, a block above n-1
 * stands for n-1, the root sends nothing (it received nothing), and a
 * processor whose to-processor is the root receives nothing.
 *
 * The operator here is the wrapping 64-bit sum; processor a contributes
 * value[b * p + a] to block b (overwritten with the partial results).
 * result[b]: the root's value of block b after the last round.
 * A partial result is combined only if the receiver expects exactly the block
 * the sender sends and has not passed its own partial result of it on yet.
 * stats[0] receiver expects a block, sender sends another one or nothing
 * stats[1] matching block, but the receiver has sent (or is sending) its partial result of it
 * stats[2] a processor sends a block it has sent before
 * stats[3] a block is sent to a processor that expects nothing
 * stats[4] (non-root processor, block) pairs whose partial result was not sent exactly once
 * stats[5] table entries outside [-q, q-1]
 * stats[6] partial results combined
 * stats[7] unused (0)
 */
int oracle_simulate_reduce(int64_t p, int64_t root, int64_t n,
                           const int32_t *recv_tab, const int32_t *send_tab,
                           uint64_t *value, uint64_t *result, uint64_t *stats)
{
    int q = oracle_q(p);
    int64_t skip[ORACLE_MAXQ + 2];
    int64_t x, i, a, b;
    int64_t *wire;
    uint64_t *wire_val;
    int32_t *times_sent;
    int k;
    if (q < 0 || n < 1 || root < 0 || root >= p) return -1;
    memset(stats, 0, 8 * sizeof(uint64_t));
    if (q == 0) { for (b = 0; b < n; b++) result[b] = value[b]; return 0; }
    oracle_skips(p, skip);
    x = (q - (n - 1) % q) % q;
    wire = (int64_t *)malloc((size_t)p * sizeof(int64_t));
    wire_val = (uint64_t *)malloc((size_t)p * sizeof(uint64_t));
    times_sent = (int32_t *)calloc((size_t)p * n, sizeof(int32_t));
    if (!wire || !wire_val || !times_sent) { free(wire); free(wire_val); free(times_sent); return -2; }
    for (a = 0; a < p; a++)
        for (k = 0; k < q; k++) {
            int32_t rv = recv_tab[a * q + k], sv = send_tab[a * q + k];
            if (rv < -q || rv > q - 1) stats[5]++;
            if (sv < -q || sv > q - 1) stats[5]++;
        }
    for (i = n + q - 1 + x - 1; i >= x; i--) {
        int64_t phase = i / q;
        k = (int)(i % q);
        /* the entry Algorithm 1 uses in round i: shifted by -x and one q per phase (Theorem 1) */
        for (a = 0; a < p; a++) {
            int32_t rv = recv_tab[a * q + k];
            int64_t blk = (int64_t)rv + phase * q - x;
            wire[a] = -1;
            if (a == root || rv < -q || rv > q - 1 || blk < 0) continue;
            if (blk > n - 1) blk = n - 1;
            wire[a] = blk;
            wire_val[a] = value[blk * p + a];
            if (times_sent[blk * p + a] > 0) stats[2]++;
        }
        for (a = 0; a < p; a++) {
            int64_t t = (a + skip[k]) % p;
            int32_t sv = send_tab[a * q + k];
            int64_t want = (int64_t)sv + phase * q - x;
            if (sv < -q || sv > q - 1 || want < 0 || t == root) want = -1;
            else if (want > n - 1) want = n - 1;
            if (want < 0) {
                if (t != root && wire[t] >= 0) stats[3]++;
            } else if (wire[t] != want) {
                stats[0]++;
            } else if (a != root && (times_sent[want * p + a] > 0 || wire[a] == want)) {
                stats[1]++;                        /* it would never be passed on */
            } else {
                value[want * p + a] += wire_val[t];
                stats[6]++;
            }
        }
        /* the sends of this round are now in the past */
        for (a = 0; a < p; a++)
            if (wire[a] >= 0) times_sent[wire[a] * p + a]++;
    }
    for (b = 0; b < n; b++) {
        result[b] = value[b * p + root];
        for (a = 0; a < p; a++)
            if (a != root && times_sent[b * p + a] != 1) stats[4]++;
    }
    free(wire); free(wire_val); free(times_sent);
    return q;
}

/*
 * Tables of Algorithm 7 for every processor: recvs[r][j][k], sends[r][j][k] for
 * processor r and root j.  With recv0/send0 == NULL they come from
 * oracle_allbroadcast_schedule, processor by processor, as the algorithm prints
 * them.  Otherwise processor r's row for root j is row (r - j) mod p of the
 * given root-0 broadcast tables (which is what the printed loops amount to; the
 * tests pin that equality), so that damaged tables can be tried.
 */
static int all_tables_(int64_t p, int q, const int32_t *recv0, const int32_t *send0,
                       int32_t **recvs_out, int32_t **sends_out)
{
    int64_t r, j;
    int k;
    size_t cells = (size_t)p * (size_t)p * (size_t)q;
    int32_t *recvs = (int32_t *)malloc(cells * sizeof(int32_t) + 1);
    int32_t *sends = (int32_t *)malloc(cells * sizeof(int32_t) + 1);
    if (!recvs || !sends) { free(recvs); free(sends); return -2; }
    for (r = 0; r < p; r++) {
        if (recv0 == NULL || send0 == NULL) {
            if (oracle_allbroadcast_schedule(p, r, 0, p, recvs + (size_t)r * p * q, sends + (size_t)r * p * q) < 0) {
                free(recvs); free(sends); return -1;
            }
        } else {
            for (j = 0; j < p; j++) {
                int64_t v = (r - j + p) % p;
                for (k = 0; k < q; k++) {
                    recvs[((size_t)r * p + j) * q + k] = recv0[v * q + k];
                    sends[((size_t)r * p + j) * q + k] = send0[v * q + k];
                }
            }
        }
    }
    *recvs_out = recvs;
    *sends_out = sends;
    return 0;
}

/* Block of a table entry in round i: Algorithm 7's shift by -x, one q per phase; -1: nothing. */
static int64_t round_block_(int32_t entry, int q, int64_t i, int64_t x, int64_t n)
{
    int64_t blk;
    if (entry < -q || entry > q - 1) return -1;
    blk = (int64_t)entry + (i / q) * q - x;
    if (blk < 0) return -1;
    return blk > n - 1 ? n - 1 : blk;
}

/*
 * Algorithm 7 run by all p processors in lock-step: every processor is the root
 * of a broadcast of its own n blocks, all p broadcasts share the rounds.  In
 * round i (k = i mod q) processor r packs, for every root j but its
 * to-processor t = (r + skip[k]) mod p, block sendblocks[j][k]; after the
 * exchange it unpacks, for every root j but itself, block recvblocks[j][k] from
 * what its from-processor f = (r - skip[k]) mod p packed for root j.  Negative
 * blocks are not packed or unpacked, a block above n-1 stands for n-1.
 *
 * arrival[(j * n + b) * p + r]: the round (from 1) in which processor r got
 * block b of root j; 0 for r = j; -1 if never.  A block is delivered only if
 * the sender packed exactly the block the receiver unpacks for that root, held
 * it before the round, and the receiver does not hold it yet.
 * stats[0..7] as for oracle_simulate_broadcast, summed over all roots.
 */
int oracle_simulate_allbroadcast(int64_t p, int64_t n, const int32_t *recv0, const int32_t *send0,
                                 int32_t *arrival, uint64_t *stats)
{
    int q = oracle_q(p);
    int64_t skip[ORACLE_MAXQ + 2];
    int64_t x, i, r, j, b;
    int32_t *recvs = NULL, *sends = NULL;
    int64_t *wire;
    unsigned char *wire_held;
    int k, rc;
    if (q < 0 || n < 1) return -1;
    memset(stats, 0, 8 * sizeof(uint64_t));
    for (j = 0; j < p; j++)
        for (b = 0; b < n; b++)
            for (r = 0; r < p; r++) arrival[(j * n + b) * p + r] = (r == j) ? 0 : -1;
    if (q == 0) return 0;
    oracle_skips(p, skip);
    rc = all_tables_(p, q, recv0, send0, &recvs, &sends);
    if (rc < 0) return rc;
    wire = (int64_t *)malloc((size_t)p * p * sizeof(int64_t));
    wire_held = (unsigned char *)malloc((size_t)p * p);
    if (!wire || !wire_held) { free(recvs); free(sends); free(wire); free(wire_held); return -2; }
    for (r = 0; r < p; r++)
        for (j = 0; j < p; j++)
            for (k = 0; k < q; k++) {
                int32_t rv = recvs[((size_t)r * p + j) * q + k], sv = sends[((size_t)r * p + j) * q + k];
                if (rv < -q || rv > q - 1) stats[5]++;
                if (sv < -q || sv > q - 1) stats[5]++;
            }
    x = (q - (n - 1) % q) % q;
    for (i = x; i < n + q - 1 + x; i++) {
        int64_t round = i - x + 1;
        k = (int)(i % q);
        /* pack: from what every processor held before the round */
        for (r = 0; r < p; r++) {
            int64_t t = (r + skip[k]) % p;
            for (j = 0; j < p; j++) {
                int64_t blk = -1;
                if (j != t) blk = round_block_(sends[((size_t)r * p + j) * q + k], q, i, x, n);
                wire[r * p + j] = blk;
                wire_held[r * p + j] = (blk >= 0 && arrival[(j * n + blk) * p + r] >= 0);
            }
        }
        /* unpack */
        for (r = 0; r < p; r++) {
            int64_t f = (r - skip[k] + p) % p;
            for (j = 0; j < p; j++) {
                int64_t want;
                if (j == r) continue;
                want = round_block_(recvs[((size_t)r * p + j) * q + k], q, i, x, n);
                if (want < 0) {
                    if (wire[f * p + j] >= 0) stats[3]++;
                } else if (wire[f * p + j] != want) {
                    stats[0]++;
                } else if (!wire_held[f * p + j]) {
                    stats[1]++;
                } else if (arrival[(j * n + want) * p + r] >= 0) {
                    stats[2]++;
                } else {
                    arrival[(j * n + want) * p + r] = (int32_t)round;
                    stats[6]++;
                    stats[7] = (uint64_t)round;
                }
            }
        }
    }
    for (j = 0; j < p; j++)
        for (b = 0; b < n; b++)
            for (r = 0; r < p; r++)
                if (arrival[(j * n + b) * p + r] < 0) stats[4]++;
    free(recvs); free(sends); free(wire); free(wire_held);
    return q;
}

/*
 * The all-reduction of Observation 1 (item 4): Algorithm 7's rounds taken from
 * the last to the first with every communication reversed, all p reductions
 * sharing the rounds.  In the round that is all-broadcast round i, processor r
 * packs, for every root j but itself, its partial result of block
 * recvblocks[j][k] and sends the message to its from-processor f; from its
 * to-processor t it receives, for every root j but t, a partial result of block
 * sendblocks[j][k], which it adds to its own.  Negative blocks move nothing, a
 * block above n-1 stands for n-1.
 *
 * value[(j * n + b) * p + r]: processor r's contribution to block b of root j
 * (overwritten with partial results); the operator is the wrapping 64-bit sum.
 * result[j * n + b]: root j's value of its block b after the last round, the
 * sum over all processors for correct tables.  A partial result is combined
 * only if the receiver expects exactly the block the sender packed for that
 * root and has not passed (and is not passing) its own partial result of it on.
 * stats[0..7] as for oracle_simulate_reduce, summed over all roots.
 */
int oracle_simulate_allreduce(int64_t p, int64_t n, const int32_t *recv0, const int32_t *send0,
                              uint64_t *value, uint64_t *result, uint64_t *stats)
{
    int q = oracle_q(p);
    int64_t skip[ORACLE_MAXQ + 2];
    int64_t x, i, r, j, b;
    int32_t *recvs = NULL, *sends = NULL;
    int64_t *wire;
    uint64_t *wire_val;
    int32_t *times_sent;
    int k, rc;
    if (q < 0 || n < 1) return -1;
    memset(stats, 0, 8 * sizeof(uint64_t));
    if (q == 0) { for (b = 0; b < n; b++) result[b] = value[b]; return 0; }
    oracle_skips(p, skip);
    rc = all_tables_(p, q, recv0, send0, &recvs, &sends);
    if (rc < 0) return rc;
    wire = (int64_t *)malloc((size_t)p * p * sizeof(int64_t));
    wire_val = (uint64_t *)malloc((size_t)p * p * sizeof(uint64_t));
    times_sent = (int32_t *)calloc((size_t)p * p * n, sizeof(int32_t));
    if (!wire || !wire_val || !times_sent) {
        free(recvs); free(sends); free(wire); free(wire_val); free(times_sent);
        return -2;
    }
    for (r = 0; r < p; r++)
        for (j = 0; j < p; j++)
            for (k = 0; k < q; k++) {
                int32_t rv = recvs[((size_t)r * p + j) * q + k], sv = sends[((size_t)r * p + j) * q + k];
                if (rv < -q || rv > q - 1) stats[5]++;
                if (sv < -q || sv > q - 1) stats[5]++;
            }
    x = (q - (n - 1) % q) % q;
    for (i = n + q - 1 + x - 1; i >= x; i--) {
        k = (int)(i % q);
        /* pack: every processor's partial results as they are before the round */
        for (r = 0; r < p; r++)
            for (j = 0; j < p; j++) {
                int64_t blk = -1;
                if (j != r) blk = round_block_(recvs[((size_t)r * p + j) * q + k], q, i, x, n);
                wire[r * p + j] = blk;
                if (blk >= 0) {
                    wire_val[r * p + j] = value[(j * n + blk) * p + r];
                    if (times_sent[(j * n + blk) * p + r] > 0) stats[2]++;
                }
            }
        /* unpack and combine */
        for (r = 0; r < p; r++) {
            int64_t t = (r + skip[k]) % p;
            for (j = 0; j < p; j++) {
                int64_t want = -1;
                if (j != t) want = round_block_(sends[((size_t)r * p + j) * q + k], q, i, x, n);
                if (want < 0) {
                    if (j != t && wire[t * p + j] >= 0) stats[3]++;
                } else if (wire[t * p + j] != want) {
                    stats[0]++;
                } else if (r != j && (times_sent[(j * n + want) * p + r] > 0 || wire[r * p + j] == want)) {
                    stats[1]++;
                } else {
                    value[(j * n + want) * p + r] += wire_val[t * p + j];
                    stats[6]++;
                }
            }
        }
        for (r = 0; r < p; r++)
            for (j = 0; j < p; j++)
                if (wire[r * p + j] >= 0) times_sent[(j * n + wire[r * p + j]) * p + r]++;
    }
    for (j = 0; j < p; j++)
        for (b = 0; b < n; b++) {
            result[j * n + b] = value[(j * n + b) * p + j];
            for (r = 0; r < p; r++)
                if (r != j && times_sent[(j * n + b) * p + r] != 1) stats[4]++;
        }
    free(recvs); free(sends); free(wire); free(wire_val); free(times_sent);
    return q;
}
