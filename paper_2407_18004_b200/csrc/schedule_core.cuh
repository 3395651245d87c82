// Per-rank schedule computation: Algorithms 2-6 of arXiv 2407.18004 restated for
// one GPU thread per rank, all state in registers.
//
// What differs from the paper's sequential formulation (results are identical):
//  * skip[k] is not stored: repeated ceil-halving composes to
//    skip[k] = ((p-1) >> (q-k)) + 1, two ALU operations.
//  * Algorithm 5's doubly linked list over the indices -1..q becomes a 32-bit set
//    (q <= 31): "next smaller remaining index" is find-highest-set-bit below e,
//    unlinking clears a bit.
//  * Algorithm 4's recursion becomes a loop.  k and s behave as globals (k is
//    returned by every call, and a caller never compares against s between a
//    callee's return and its own next assignment to s), and the indices of the
//    pending calls strictly decrease with depth, so the call stack is a second
//    32-bit set and r' is the sum of its skips; "return" pops the lowest set bit.
//    The callee's first test of the index its caller just used can never pass and
//    is skipped.
//  * Positions are kept as distances from the target R = p + r:
//    u = R - r', v = R - s.  The tests of Algorithm 4 become
//      r'+skip[e] <= R-skip[k]    <=>  skip[e] + skip[k]   <= u
//      r'+skip[e] <  s            <=>  skip[e] + v         <  u
//      r'+skip[e] <= R-skip[k+1]  <=>  skip[e] + skip[k+1] <= u
//      r' > R-skip[k+1]           <=>  u < skip[k+1]
//    and every quantity stays below 2^32 for p up to 2^31-1 (r'+skip[e] itself
//    can reach 3p).  The initial s = 2p can never fail its test, so v starts at 0.
#pragma once
#include <stdint.h>

namespace bcast {

struct Geometry {
    uint32_t p;     // number of processors, 2 <= p <= 2^31-1
    uint32_t pm1;   // p - 1
    int      q;     // ceil(log2 p), 1..31
};

__device__ __forceinline__ Geometry make_geometry(uint32_t p)
{
    Geometry g;
    g.p = p;
    g.pm1 = p - 1u;
    g.q = 32 - __clz(p - 1u);          // p >= 2
    return g;
}

// Algorithm 2 in closed form; valid for 0 <= k <= q.
__host__ __device__ __forceinline__ uint32_t skip_of(const Geometry &g, int k)
{
    return (g.pm1 >> (g.q - k)) + 1u;
}

// Index of the highest set bit of x != 0.
__host__ __device__ __forceinline__ int top_bit(uint32_t x)
{
#ifdef __CUDA_ARCH__
    return 31 - __clz(x);
#else
    return 31 - __builtin_clz(x);
#endif
}

// Algorithm 3: smallest index of the canonical skip sequence of r; q for r = 0.
__device__ __forceinline__ int baseblock(const Geometry &g, uint32_t r)
{
    uint32_t rem = r;                  // r - r'
    for (int k = g.q - 1; k >= 0; --k) {
        const uint32_t s = skip_of(g, k);
        if (s == rem) return k;
        if (s < rem) rem -= s;
    }
    return g.q;
}

// Counters the verification sweep reads; the table kernels pass a dummy.
struct SearchStats {
    int descents;       // recursive calls of Algorithm 4 in the current search
    int steps;          // list elements examined in the current search (Lemma 6 counts these)
    int capped;         // some search hit the loop's safety cap
    int over_bound;     // some search exceeded q-1 descents or 2q+R steps (Lemmas 5, 6)
};

struct NoStats {
    __host__ __device__ __forceinline__ void begin() {}
    __host__ __device__ __forceinline__ void descent() {}
    __host__ __device__ __forceinline__ void step() {}
    __host__ __device__ __forceinline__ void cap() {}
    __host__ __device__ __forceinline__ void end(int) {}
    __host__ __device__ __forceinline__ void violation(uint32_t, int) {}
};

struct CountStats {
    SearchStats s{0, 0, 0, 0};
    uint32_t *row_violations = nullptr;     // per tile row: rounds another lane found undecided in Algorithm 6
    __device__ __forceinline__ void violation(uint32_t row, int k)
    { if (row_violations) atomicOr(row_violations + row, 1u << k); }
    __device__ __forceinline__ void begin() { s.descents = 0; s.steps = 0; }
    __device__ __forceinline__ void descent() { s.descents++; }
    __device__ __forceinline__ void step() { s.steps++; }
    __device__ __forceinline__ void cap() { s.capped = 1; }
    __device__ __forceinline__ void end(int q)
    { if (s.descents > q - 1 || s.steps > 2 * q + s.descents) s.over_bound = 1; }
};

// Value emitted for the rounds a search did not reach because it ran into its iteration cap
// (BCAST_UNRESOLVED in the public header).  The cap lies far above Lemma 6's bound; no p is
// known to reach it.
constexpr int kUnresolvedEntry = -128;

// State of the search of Algorithm 4 between two loop iterations.
struct SearchState {
    uint32_t remaining;   // list of skip indices still linked
    uint32_t pending;     // indices of the calls in progress (the recursion stack)
    uint32_t cand;        // part of the list the current call still has to scan
    uint32_t u;           // R - r'
    int b;                // baseblock of the rank
    int k = 0;            // round the search is in (entries accepted so far)
    uint32_t v = 0;       // R - s, s the processor accepted last (0 before the first: s = 2p never binds)
};

// Algorithm 5's set-up: all indices 0..q but the baseblock b, r' = 0, e = q.
__device__ __forceinline__ SearchState search_from_top(const Geometry &g, uint32_t r, int b)
{
    SearchState s;
    s.remaining = ((2u << g.q) - 1u) & ~(1u << b);
    s.pending = 0u;
    s.cand = s.remaining;
    s.u = g.p + r;
    s.b = b;
    return s;
}

// The same search, entered where its first run of recursive calls ends.  While k = 0
// the search descends on an index e exactly when skip[e] + 2 <= R - r', and R - r' is
// then the part of R = p + r that the greedy decomposition of R over the skips
// (skip[q] = p first) has not covered yet: every digit is descended on as long as at
// least 2 remains after it, and every non-digit fails its test.  The walk below finds
// that point with one compare per level instead of one search step, and the baseblock
// on the way: the digit that leaves 0 is the baseblock (it is not in the list, the scan
// goes on below it); a digit that leaves 1 is followed by digit 0 only, so the
// baseblock is 0 and that digit is the next candidate.  The skipped steps and descents
// are added to the counters so that the bounds of Lemmas 5 and 6 are still checked
// against the whole search.
template <class Stats>
__device__ __forceinline__ SearchState search_from_digits(const Geometry &g, uint32_t r, Stats &stats)
{
    SearchState s;
    uint32_t rem = g.p + r;
    s.pending = 0u;
    int k = g.q;
    int b = 0;
    // ends at level 1 at the latest (the remainder entering level k is below skip[k+1], so it is 2
    // or 3 there); the bound on k only keeps the loop finite whatever happens
    for (; k > 0; --k) {
        const uint32_t sk = skip_of(g, k);
        if (rem >= sk) {
            const uint32_t left = rem - sk;
            if (left < 2u) { b = left == 0u ? k : 0; break; }
            s.pending |= 1u << k;
            rem = left;
            stats.descent();
        }
        stats.step();
    }
    s.remaining = ((2u << g.q) - 1u) & ~(1u << b);
    s.cand = s.remaining & ((2u << k) - 1u);
    s.u = rem;
    s.b = b;
    return s;
}

// Algorithms 4 and 5 from a given state (k = 0, nothing accepted yet).  emit(k, value)
// is called once for each k = 0..k_last in increasing order with the final schedule
// value (b where the search accepted index q, else index - q).  k_last = q-1 yields
// the whole row; a smaller k_last stops early.
template <class Emit, class Stats>
__host__ __device__ __forceinline__ void recv_search_run(const Geometry &g, const SearchState &st, int k_last,
                                                Emit emit, Stats &stats)
{
    const int q = g.q;
    const int b = st.b;
    uint32_t remaining = st.remaining;
    uint32_t pending = st.pending;
    uint32_t cand = st.cand;
    uint32_t u = st.u;                                    // R - r'
    uint32_t v = st.v;                                    // R - s
    int k = st.k;
    uint32_t sk_k = skip_of(g, k);                        // skip[k]
    uint32_t sk_k1 = skip_of(g, k + 1 <= q ? k + 1 : q);  // skip[k+1]
    uint32_t m = sk_k > v + 1u ? sk_k : v + 1u;           // max(skip[k], v+1)
    int guard = 6 * q + 16;                               // never reached; keeps the loop finite

    while (true) {
        if (--guard < 0) {                                // mark what was still wanted and give up
            stats.cap();
            for (int kk = k; kk <= k_last; ++kk) emit(kk, kUnresolvedEntry);
            return;
        }
        int e;
        uint32_t bit, sk_e;
        bool accept;
        if (cand != 0u) {
            e = top_bit(cand);
            bit = 1u << e;
            cand ^= bit;
            sk_e = skip_of(g, e);
            stats.step();
            // both outer tests of Algorithm 4: skip[e] <= u - max(skip[k], v+1)
            if (u < m || sk_e > u - m) continue;
            if (sk_e + sk_k1 <= u) {                      // room for a closer processor: descend
                pending |= bit;
                u -= sk_e;
                stats.descent();
                continue;
            }
            accept = (u >= sk_k1);
            if (!accept) cand = 0u;                       // r' > R - skip[k+1]: return
        } else {
            if (pending == 0u) { stats.end(q); return; }  // outermost call ran off the list
            bit = pending & (0u - pending);               // innermost pending call
            pending ^= bit;
            e = top_bit(bit);
            sk_e = skip_of(g, e);
            u += sk_e;                                    // back in the caller's frame
            accept = (u >= sk_k1);                        // else the caller returns as well
        }
        if (accept) {
            emit(k, e == q ? b : e - q);
            if (k == k_last) { stats.end(q); return; }
            v = u - sk_e;                                 // s = r' + skip[e]
            remaining &= ~bit;
            cand = remaining & (bit - 1u);
            ++k;
            sk_k = sk_k1;
            sk_k1 = skip_of(g, k + 1 <= q ? k + 1 : q);
            m = sk_k > v + 1u ? sk_k : v + 1u;
        }
    }
}

// Algorithms 4 and 5 for virtual rank r with baseblock b, as printed: from the top.
template <class Emit, class Stats>
__device__ __forceinline__ void recv_search(const Geometry &g, uint32_t r, int b, int k_last,
                                            Emit emit, Stats &stats)
{
    stats.begin();
    recv_search_run(g, search_from_top(g, r, b), k_last, emit, stats);
}

// The same result, entered after the first run of recursive calls.  Returns the baseblock.
template <class Emit, class Stats>
__device__ __forceinline__ int recv_search_fast(const Geometry &g, uint32_t r, int k_last,
                                                Emit emit, Stats &stats)
{
    stats.begin();
    const SearchState st = search_from_digits(g, r, stats);
    recv_search_run(g, st, k_last, emit, stats);
    return st.b;
}

// Algorithm 6 for virtual rank r > 0 with baseblock b: emit(k, value) for
// k = q-1..1 and then k = 0.  Rounds the fast rules cannot decide are returned as
// a bit set (at most four by Theorem 3); the caller fills those entries with
// recvblock[k] of rank (r + skip[k]) mod p.
template <class Emit>
__device__ __forceinline__ uint32_t send_walk(const Geometry &g, uint32_t r, int b, Emit emit)
{
    const int q = g.q;
    uint32_t rp = r;            // virtual processor index r'
    uint32_t e = g.p;           // upper bound on the range of virtual processors
    int c = b;                  // block the lower part keeps sending
    uint32_t violations = 0;
    uint32_t sk = skip_of(g, q - 1);
    for (int k = q - 1; k >= 1; --k) {
        const uint32_t sk_below = skip_of(g, k - 1);
        bool viol;
        if (rp < sk) {                                    // lower part
            viol = !(rp + sk < e || e < sk_below || (k == 1 && b > 0));
            if (e > sk) e = sk;
        } else {                                          // upper part
            c = k - q;
            viol = !(k == 1 || rp > sk || e - sk < sk_below) && (rp + sk > e);
            rp -= sk;
            e -= sk;
        }
        if (viol) violations |= 1u << k;
        emit(k, c);
        sk = sk_below;
    }
    emit(0, b - q);
    return violations;
}

// One entry of another rank's receive schedule: recvblock[k] of virtual rank t.
template <class Stats>
__device__ __forceinline__ int recv_entry(const Geometry &g, uint32_t t, int k, Stats &stats)
{
    int value = 0;
    recv_search_fast(g, t, k, [&](int kk, int val) { if (kk == k) value = val; }, stats);
    return value;
}

// ---------------------------------------------------------------------------------------
// The low rounds of the search, once per low state instead of once per rank.
//
// Let u >= 2 be what is left of R = p + r after its greedy digits at the levels >= L
// (skip[q] = p first).  The search of Algorithms 4 and 5 descends on exactly those digits
// before it accepts anything (search_from_digits), and from then on, until it first
// returns past level L, every quantity it looks at is local to the levels below L: the
// distance u, the list of indices < L without the baseblock (which is the lowest digit of
// u, since u > 0), the skips below L and skip[k], skip[k+1] of the rounds it is in.  The
// indices it accepts in that stretch are therefore a function of u alone for a given p, and
// so is the number n of rounds it completes there.  When the stretch ends, the search
// returns into the call that descended on the lowest digit j >= L of R and accepts j for
// round n at once (R - r' >= skip[j] >= skip[n+1]), which gives one more round.
//
// The table of a frame packs that per u, a nibble per round k = 0..7: the accepted index
// (< L <= 14), kLowFramePop for "the lowest digit of R at or above L" (value j - q, or the
// rank's own baseblock when j = q), kLowFrameNone for rounds beyond.  u < 2 gives no rounds:
// there the search stops descending above level L.
//
// The entries are built from one another.  Let x be the highest digit of u, u' = u - skip[x].
// For u' >= 2 the search first descends on x and is then in the same situation one frame
// down, so its first rounds are the entry of u'; where that stretch ends it returns to x
// and accepts it.  (u' = 1: x is accepted for round 0 at once.  u' = 0: x is the baseblock
// and not in the list.)  Only what follows needs the search itself, started from the state
// that prefix leaves: back in the outermost call, scanning below x.  The table depends on
// p alone, so the host fills it once per launch, in increasing u (low_frame_fill), and
// hands it to the kernel among its arguments; every block copies it to shared memory.
constexpr uint32_t kLowFramePop = 14u;
constexpr uint32_t kLowFrameNone = 15u;
constexpr int kLowFrameRounds = 8;

// Entry of u, skip[x] <= u < skip[x+1], given the entries of every smaller u.
__host__ __device__ __forceinline__ uint32_t low_frame_entry(const Geometry &g, int L, const uint32_t *table,
                                                             int x, uint32_t u)
{
    constexpr uint32_t kNone = 0xffffffffu;
    if (u < 2u) return kNone;
    const uint32_t sk_x = skip_of(g, x);
    const uint32_t left = u - sk_x;                        // u'
    uint32_t packed = kNone;
    uint32_t taken = 0u;                                   // indices accepted so far
    int rounds = 0;
    int b = x;                                             // left = 0: x is the baseblock
    if (left >= 1u) {
        // the baseblock: lowest digit of u, i.e. of u'
        uint32_t rem = left;
        for (int k = x - 1; k >= 0; --k) {
            const uint32_t s = skip_of(g, k);
            if (rem >= s) { rem -= s; if (rem == 0u) { b = k; break; } }
        }
        if (left >= 2u) {
            const uint32_t prefix = table[left];
            while (rounds < kLowFrameRounds) {
                const uint32_t nib = (prefix >> (4 * rounds)) & 15u;
                if (nib >= kLowFramePop) break;
                taken |= 1u << nib;
                ++rounds;
            }
            if (rounds == kLowFrameRounds) return prefix;
            packed = prefix | (kNone << (4 * rounds));      // the prefix's rounds, nothing beyond yet
        }
        packed = (packed & ~(15u << (4 * rounds))) | ((uint32_t)x << (4 * rounds));    // x accepted
        taken |= 1u << x;
        if (++rounds == kLowFrameRounds) return packed;
    }
    SearchState s;
    s.b = b;
    s.remaining = ((1u << L) - 1u) & ~(1u << b) & ~taken;
    s.pending = 0u;
    s.cand = s.remaining & ((1u << x) - 1u);
    s.u = u;
    s.k = rounds;
    s.v = left >= 1u ? left : 0u;
    bool capped = false;
    NoStats ns;
    recv_search_run(g, s, kLowFrameRounds - 1, [&](int k, int val) {
        if (val == kUnresolvedEntry) { capped = true; return; }
        packed = (packed & ~(15u << (4 * k))) | ((uint32_t)(val + g.q) << (4 * k));
        rounds = k + 1;
    }, ns);
    if (capped) return kNone;
    if (rounds < kLowFrameRounds)
        packed = (packed & ~(15u << (4 * rounds))) | (kLowFramePop << (4 * rounds));
    return packed;
}

// Fills table[0 .. min(skip[L], capacity)), every entry from the ones before it.
inline void low_frame_fill(const Geometry &g, int L, uint32_t *table, uint32_t capacity)
{
    const uint32_t n_states = skip_of(g, L) < capacity ? skip_of(g, L) : capacity;
    for (uint32_t u = 0; u < 2u && u < n_states; ++u) table[u] = 0xffffffffu;
    for (int x = 1; x < L; ++x) {
        const uint32_t lo = skip_of(g, x);
        const uint32_t hi = skip_of(g, x + 1) < n_states ? skip_of(g, x + 1) : n_states;
        for (uint32_t u = lo; u < hi; ++u) table[u] = low_frame_entry(g, L, table, x, u);
    }
}

}  // namespace bcast
