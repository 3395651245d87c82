// Closed-form schedule rows: one pass over the levels k = q-1..0 per rank, no search.
//
// The send row is Algorithm 6 as printed.  The receive row uses correctness
// condition 1, recvblock[k]_r = sendblock[k]_f with f = (r - skip[k]) mod p, and
// evaluates Algorithm 6's round-k rule for f WITHOUT walking f's levels, from
// the state r's own walk already carries:
//
//  * Write R = p + r and treat skip[q] = p as a digit that is always set, so that
//    f = R - skip[k] needs no modulo.  The walk of Algorithm 6 over r decides at
//    each level whether r' >= skip[k] ("upper", digit k of r set) or not.
//  * Digit k set: f has the digits of r with digit k cleared; every decision of
//    f's walk above k equals r's, f is in the lower part at k, r' + skip[k] of f
//    is r's own r' < e, so the rule never reports a violation there and
//    recvblock[k] = c, the block the lower part keeps sending (the lowest set
//    digit above k, minus q); with no digit above k it is the baseblock of r.
//  * Digit k clear: subtracting skip[k] borrows from the lowest set digit j above
//    k.  f's walk equals r's above j, is in the lower part at j, and below j it
//    is in the upper part at every level down to k+1 exactly when
//        X = r'_j - skip[k] - (skip[k+1] + ... + skip[j-1])  >= 0,
//    r'_j being r's virtual index entering level j; X is then f's virtual index
//    entering level k and min(e_j, skip[j]) - (same sum) its bound, which is all
//    round k's rule needs.  With below[l] = skip[0] + ... + skip[l-1] this is
//        X = (r'_j - below[j]) + below[k],   bound = (min(e_j, skip[j]) - below[j]) + below[k+1],
//    so two registers saved at level j serve every k below it.
//  * Whenever the rule reports a violation for (f, k), or X < 0, or the value
//    would be a baseblock this pass cannot know, the entry is flagged and the
//    caller computes it with the search of Algorithms 4 and 5.
//
// Q is a template parameter so that the level loop unrolls completely: skips and
// prefix sums become constant-bank operands and row offsets immediates.  The
// violation tests are split into a cheap necessary condition in the hot path and
// the full rule behind a rarely taken branch.
#pragma once
#include <stdint.h>

namespace bcast {

struct LevelTables {
    uint32_t skip[33];      // skip[0..q]
    uint32_t below[34];     // below[l] = skip[0] + ... + skip[l-1]
};

constexpr int kMarkBase = 100;      // stands for "the baseblock of r" until it is known

template <int Q> struct WalkInt { typedef int32_t type; };      // p <= 2^30: p + r < 2^31
template <> struct WalkInt<31> { typedef int64_t type; };

// State of Algorithm 6's walk over r between two levels, with what the receive rule needs.
template <class Int>
struct WalkState {
    Int rp;     // virtual processor index r'
    Int e;      // bound on the virtual range
    Int A;      // r'_j - below[j], j the lowest upper level so far (j = q, r' = p + r at first)
    Int E;      // min(e_j, skip[j]) - below[j]
    int c;      // block the lower part sends
    int cJ;     // c entering level j
    int j;
};

template <int Q>
__device__ __forceinline__ WalkState<typename WalkInt<Q>::type> walk_start(const LevelTables &tab, uint32_t p,
                                                                          uint32_t r)
{
    typedef typename WalkInt<Q>::type Int;
    WalkState<Int> s;
    s.rp = (Int)r;
    s.e = (Int)p;
    s.A = (Int)p + (Int)r - (Int)tab.below[Q];
    s.E = (Int)p - (Int)tab.below[Q];
    s.c = kMarkBase;
    s.cJ = kMarkBase;
    s.j = Q;
    return s;
}

// Levels FROM-1 .. 0 of the pass for one rank.  Entries are written through recv_row /
// send_row; rounds the rules cannot decide are added to recv_flags / viol.
template <int Q, int FROM, class Row, class Int>
__device__ __forceinline__ void closed_form_levels(const LevelTables &tab, WalkState<Int> &s, Row recv_row,
                                                   Row send_row, uint32_t &recv_flags, uint32_t &viol)
{
    Int rp = s.rp, e = s.e, A = s.A, E = s.E;
    int c = s.c, cJ = s.cJ, j = s.j;
#pragma unroll
    for (int k = FROM - 1; k >= 0; --k) {
        const Int sk = (Int)tab.skip[k];
        const Int sk_below = k > 0 ? (Int)tab.skip[k - 1] : 0;
        if (rp >= sk) {                                              // upper part: digit k set
            recv_row(k, c);
            if (k > 0) {
                send_row(k, k - Q);
                // a violation needs r' = skip[k]
                if (k > 1 && rp == sk && e - sk >= sk_below && rp + sk > e) viol |= 1u << k;
            }
            A = rp - (Int)tab.below[k];
            E = min(e, sk) - (Int)tab.below[k];
            cJ = c;
            j = k;
            c = k - Q;
            rp -= sk;
            e -= sk;
        } else {                                                     // lower part: digit k clear
            if (k > 0) {
                send_row(k, c);
                // a violation needs r' + skip[k] >= e
                if (rp + sk >= e && !(e < sk_below || (k == 1 && rp == 0))) viol |= 1u << k;
            }
            // round-k rule of Algorithm 6 for f = R - skip[k]
            const Int X = A + (Int)tab.below[k];
            const Int eB = E + (Int)tab.below[k + 1];
            const bool upB = X >= sk;
            recv_row(k, upB ? k - Q : (j > k + 1 ? k + 1 - Q : cJ));
            if (X < 0 || (upB ? X == sk : X + sk >= eB)) {
                const bool ok = X >= 0 && (upB ? (k <= 1 || eB - sk < sk_below || X + sk <= eB)
                                               : (k == 0 || eB < sk_below || (k == 1 && X == 0)));
                if (!ok) recv_flags |= 1u << k;
            }
            e = min(e, sk);
        }
    }
    s.rp = rp; s.e = e; s.A = A; s.E = E; s.c = c; s.cJ = cJ; s.j = j;
}

// After level 0: b is the lowest set digit of r (the last upper level).  Fills the
// entries that stand for "baseblock of r" and returns b.
template <int Q, class Row>
__device__ __forceinline__ int closed_form_finish(const LevelTables &tab, uint32_t r, int b, Row recv_row,
                                                  Row send_row, uint32_t &recv_flags)
{
    // the highest set digit is the largest k with skip[k] <= r, one of the two levels
    // around r's bit length
    const int len = 31 - __clz(r);
    const int top = len + (len + 1 < Q && r >= tab.skip[len + 1] ? 1 : 0);
    send_row(0, b - Q);
    // entries still standing for "baseblock of r": every send round above the top digit
    // and the receive entry of the top digit; one below it the receive entry may be the
    // baseblock of f, which only the search knows
    for (int k = Q - 1; k > top; --k) send_row(k, b);
    recv_row(top, b);
    if (Q > 1 && top > 0 && recv_row.get(top - 1) == kMarkBase) recv_flags |= 1u << (top - 1);
    return b;
}

// Rows of virtual rank r >= 1.  recv_row/send_row: (k, value) writers that can also
// read back an entry.  Returns the rounds whose receive entry must come from the
// search; *send_flags receives the rounds whose send entry must (Algorithm 6's
// violations) and *baseblock_out the baseblock of r.
template <int Q, class Row>
__device__ __forceinline__ uint32_t closed_form_rows(const LevelTables &tab, uint32_t p, uint32_t r,
                                                     Row recv_row, Row send_row, uint32_t *send_flags,
                                                     int *baseblock_out)
{
    uint32_t recv_flags = 0, viol = 0;
    auto s = walk_start<Q>(tab, p, r);
    closed_form_levels<Q, Q>(tab, s, recv_row, send_row, recv_flags, viol);
    *baseblock_out = closed_form_finish<Q>(tab, r, s.j, recv_row, send_row, recv_flags);
    *send_flags = viol;
    return recv_flags;
}

// ---------------------------------------------------------------------------------------
// Sharing the high levels among the ranks of a tile.
//
// The ranks r_first .. r_first+rows-1 of a tile (consecutive, none of them the root, no
// wrap past p-1) fall into a few RUNS that agree on their digits at the levels from
// kSharedFrom up: a run ends where a clear digit's remainder reaches its skip, so its
// length is the minimum over the clear levels of skip[k] - r'_k.  Within a run everything
// the rules look at is the base rank's value plus the offset t of the rank in the run:
// r'_k(t) = r'_k + t, A(t) = A + t, while e, E, c, cJ and j do not depend on t.  Hence
//   * an upper level's entries are constants, with a violation possible only at the one
//     offset where r'_k(t) = skip[k];
//   * a lower level's send entry is constant and its receive entry switches once, at
//     the offset where X(t) = X + t reaches skip[k]; the necessary conditions for
//     "undecided" are intervals of t.
// One warp builds these descriptions for a whole tile, with one LANE PER LEVEL (lane l
// owns level kSharedFrom-1+l; lane 0's level is the first one that is walked per rank and
// only its entering state is kept).  Every rank of the tile then copies its high-level
// entries from the description of its run and walks only the levels below kSharedFrom.
//
// build_tile_runs:
//  step 1 (all lanes, same work): walk the base rank's digits from q-1 down to kSharedFrom;
//          each lane keeps r' and e as they were entering its level;
//  step 2 (lane per level): c and j from the digit set by bit scans; A, E from the lane that
//          owns level j (two shuffles);
//  step 3 (lane per level): the level's entry values and switch offset; the full rules are
//          evaluated inside the suspicious intervals (rare) and undecided entries are noted
//          in the tile's pending list.
constexpr int kSharedFrom = 9;
// A run is as long as there are values of the remainder below kSharedFrom for its digits: at least
// skip[kSharedFrom] - 1 >= 2^(kSharedFrom-1) = kThreads ranks, so a tile of kThreads rows meets at most one
// boundary between runs.  (A tile that would need more is given up and walked rank by rank.)
constexpr int kMaxRuns = 2;
constexpr int kMaxPending = 32;
constexpr int kSharedLevels = 31 - kSharedFrom;         // most levels a description can hold

template <class Int>
struct TileRuns {
    int n_runs;                             // 0: no description, walk every level per rank
    int n_pending;
    int start[kMaxRuns + 1];                // first row of each run; unused entries hold the row count
    WalkState<Int> state[kMaxRuns];         // entering level kSharedFrom-1, for the run's base rank
    uint32_t level[kMaxRuns][kSharedLevels];   // send entry | receive entry before the switch << 8 | switch offset << 16;
                                               // from the switch on the receive entry is k - q
    uint32_t pending[kMaxPending];          // row | k << 9 | is_send << 14
    uint32_t full_len[kMaxRuns];            // ranks from the run's first row on that share its digits and lie below p,
                                            // also past the tile's end
};

// Executed by one whole warp.  tab: uniform-index tables; lookup: tables for per-lane indices.
template <int Q>
__device__ __forceinline__ void build_tile_runs(const LevelTables &tab, const LevelTables &lookup, uint32_t p,
                                                uint32_t r_first, int rows, int lane,
                                                TileRuns<typename WalkInt<Q>::type> &out)
{
    typedef typename WalkInt<Q>::type Int;
    constexpr unsigned kFull = 0xffffffffu;
    const int my = kSharedFrom - 1 + lane;          // the level this lane owns
    const bool owner = my < Q;
    const bool column = owner && my >= kSharedFrom;
    const int k = column ? my : kSharedFrom;        // keeps idle lanes' table indices in range
    const Int sk = (Int)lookup.skip[k];
    const Int sk_below = (Int)lookup.skip[k - 1];
    int n_runs = 0;
    bool give_up = false;
    if (lane == 0) out.n_pending = 0;
    __syncwarp();

    int ib = 0;                                     // first row of the current run
    while (ib < rows && !give_up) {
        if (n_runs == kMaxRuns) { give_up = true; break; }
        // ---- step 1: digits of the base rank, the same in every lane
        const uint32_t base = r_first + (uint32_t)ib;
        Int rem = (Int)base;
        Int e = (Int)p;
        uint32_t digits = 0;
        Int my_rp = 0, my_e = 0;
#pragma unroll
        for (int kk = Q - 1; kk >= kSharedFrom; --kk) {
            if (kk == my) { my_rp = rem; my_e = e; }
            const Int s = (Int)tab.skip[kk];
            if (rem >= s) {
                rem -= s;
                e -= s;
                digits |= 1u << kk;
            } else {
                e = min(e, s);
            }
        }
        if (my == kSharedFrom - 1) { my_rp = rem; my_e = e; }
        const bool upper = column && ((digits >> k) & 1u);
        // the run ends where a clear digit's remainder reaches its skip
        Int run = column && !upper ? sk - my_rp : (Int)0x7fffffff;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) run = min(run, __shfl_xor_sync(kFull, run, off));
        const int n = (int)min(run, (Int)(rows - ib));          // rows ib .. ib+n-1
        if (lane == 0) out.full_len[n_runs] = (uint32_t)min(run, (Int)p - (Int)base);

        // ---- step 2: what level `my` sees above it
        const uint32_t above = owner ? digits >> (my + 1) : 0u;
        const int j = above != 0u ? my + __ffs(above) : Q;      // lowest set digit above my level
        const int c = j < Q ? j - Q : kMarkBase;
        const int jl = j < Q ? j - (kSharedFrom - 1) : 0;       // lane that owns level j
        const Int rp_j = __shfl_sync(kFull, my_rp, jl);
        const Int e_j = __shfl_sync(kFull, my_e, jl);
        Int A, E;
        int cJ;
        if (j < Q) {
            const uint32_t above_j = digits >> (j + 1);
            const int jj = above_j != 0u ? j + __ffs(above_j) : Q;
            cJ = jj < Q ? jj - Q : kMarkBase;
            A = rp_j - (Int)lookup.below[j];
            E = min(e_j, (Int)lookup.skip[j]) - (Int)lookup.below[j];
        } else {
            cJ = kMarkBase;
            A = (Int)p + (Int)base - (Int)lookup.below[Q];
            E = (Int)p - (Int)lookup.below[Q];
        }
        if (lane == 0) {
            WalkState<Int> s;
            s.rp = my_rp; s.e = my_e; s.A = A; s.E = E; s.c = c; s.cJ = cJ; s.j = j;
            out.state[n_runs] = s;
            out.start[n_runs] = ib;
        }

        // ---- step 3: level `my` for offsets t = 0 .. n-1 of this run
        if (column) {
            int send_v, recv_v0;
            Int t_switch;                                       // receive entry is k - q from this offset on
            Int s_lo, s_hi, r_lo, r_hi;                         // suspicious offsets [lo, hi)
            Int X = 0, eB = 0;
            if (upper) {
                send_v = k - Q;
                recv_v0 = c;
                t_switch = 0;
                const Int t_eq = sk - my_rp;                    // where r'(t) = skip[k]
                const bool possible = my_e - sk >= sk_below && sk + sk > my_e;
                s_lo = possible ? t_eq : (Int)n;
                s_hi = possible ? t_eq + 1 : (Int)n;
                r_lo = r_hi = (Int)n;
            } else {
                send_v = c;
                s_lo = my_e < sk_below ? (Int)n : my_e - sk - my_rp;   // r'(t) + skip[k] >= e
                s_hi = (Int)n;
                X = A + (Int)lookup.below[k];                   // f's virtual index entering level k at t = 0
                eB = E + (Int)lookup.below[k + 1];
                recv_v0 = j > k + 1 ? k + 1 - Q : cJ;
                t_switch = sk - X;
                // X(t) < 0, X(t) = skip[k], and X(t) + skip[k] >= eB below the switch all lie in
                // one interval that ends at the switch; the full rule is evaluated inside it
                const Int t_low = eB - sk - X;                  // first t with X(t) + skip[k] >= eB
                if (X >= 0 && eB < sk_below) {
                    r_lo = r_hi = (Int)n;                       // the rule accepts every offset
                } else {
                    r_lo = X < 0 ? (Int)0 : min(t_low, t_switch);
                    r_hi = t_switch + 1;
                }
            }
            // an upper level never switches; a lower level switches to recv_v1 = k - q
            const Int ts = upper ? (Int)0xffff : max((Int)0, min(t_switch, (Int)rows));
            out.level[n_runs][k - kSharedFrom] =
                (uint32_t)(send_v & 0xff) | ((uint32_t)(recv_v0 & 0xff) << 8) | ((uint32_t)ts << 16);
            // undecided entries: the full rules, only inside the intervals found above
            const Int s_from = max(s_lo, (Int)0), s_to = min(s_hi, (Int)n);
            for (Int t = s_from; t < s_to; ++t) {
                const Int rp_t = my_rp + t;
                const bool bad = upper ? (rp_t == sk && my_e - sk >= sk_below && rp_t + sk > my_e)
                                       : (rp_t + sk >= my_e && !(my_e < sk_below));
                if (bad) {
                    const int slot = atomicAdd(&out.n_pending, 1);
                    if (slot < kMaxPending) out.pending[slot] = (uint32_t)(ib + (int)t) | ((uint32_t)k << 9) | (1u << 14);
                }
            }
            const Int r_from = max(r_lo, (Int)0), r_to = min(r_hi, (Int)n);
            for (Int t = r_from; t < r_to; ++t) {
                const Int Xt = X + t;
                const bool upB = Xt >= sk;
                if (Xt < 0 || (upB ? Xt == sk : Xt + sk >= eB)) {
                    const bool ok = Xt >= 0 && (upB ? (eB - sk < sk_below || Xt + sk <= eB) : (eB < sk_below));
                    if (!ok) {
                        const int slot = atomicAdd(&out.n_pending, 1);
                        if (slot < kMaxPending) out.pending[slot] = (uint32_t)(ib + (int)t) | ((uint32_t)k << 9);
                    }
                }
            }
        }
        ib += n;
        ++n_runs;
    }
    __syncwarp();
    if (lane == 0) {
        const bool usable = !give_up && out.n_pending <= kMaxPending;
        out.n_runs = usable ? n_runs : 0;
        if (!usable) out.n_pending = 0;
        for (int i = usable ? n_runs : 0; i <= kMaxRuns; ++i) out.start[i] = rows;
    }
}

// The high-level entries of the rank in row `row` from its run's description; returns
// the walk state entering level kSharedFrom-1 for that rank and, on request, the first row
// past the rank's run.
template <int Q, class Row>
__device__ __forceinline__ WalkState<typename WalkInt<Q>::type>
apply_tile_runs(const TileRuns<typename WalkInt<Q>::type> &runs, int row, Row recv_row, Row send_row,
                int *run_end = nullptr)
{
    typedef typename WalkInt<Q>::type Int;
    int run = 0;
#pragma unroll
    for (int i = 1; i < kMaxRuns; ++i) run += row >= runs.start[i] ? 1 : 0;
    const int t = row - runs.start[run];
    if (run_end != nullptr) *run_end = runs.start[run + 1];     // unused entries hold the row count
    WalkState<Int> s = runs.state[run];
    s.rp += (Int)t;
    s.A += (Int)t;
#pragma unroll
    for (int k = Q - 1; k >= kSharedFrom; --k) {
        const uint32_t d = runs.level[run][k - kSharedFrom];
        send_row(k, (int)d);                               // the writers keep the low byte
        recv_row(k, (uint32_t)t >= (d >> 16) ? k - Q : (int)(d >> 8));
    }
    return s;
}

}  // namespace bcast
