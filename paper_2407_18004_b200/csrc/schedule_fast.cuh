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

// Rows of virtual rank r >= 1.  recv_row/send_row: (k, value) writers that can also
// read back an entry.  Returns the rounds whose receive entry must come from the
// search; *send_flags receives the rounds whose send entry must (Algorithm 6's
// violations) and *baseblock_out the baseblock of r.
template <int Q, class Row>
__device__ __forceinline__ uint32_t closed_form_rows(const LevelTables &tab, uint32_t p, uint32_t r,
                                                     Row recv_row, Row send_row, uint32_t *send_flags,
                                                     int *baseblock_out)
{
    typedef typename WalkInt<Q>::type Int;
    Int rp = (Int)r;                 // Algorithm 6: virtual processor index r'
    Int e = (Int)p;                  //              bound on the virtual range
    int c = kMarkBase;               //              block the lower part sends
    // saved at the lowest upper level j seen so far (j = q at first, r' = p + r, e = p)
    Int A = (Int)p + (Int)r - (Int)tab.below[Q];    // r'_j - below[j]
    Int E = (Int)p - (Int)tab.below[Q];             // min(e_j, skip[j]) - below[j]
    int cJ = kMarkBase;                             // c entering level j
    int j = Q;
    uint32_t recv_flags = 0, viol = 0;

#pragma unroll
    for (int k = Q - 1; k >= 0; --k) {
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
    // j is now the lowest set digit of r, its baseblock; the highest set digit is the
    // largest k with skip[k] <= r, one of the two levels around r's bit length
    const int b = j;
    const int len = 31 - __clz(r);
    const int top = len + (len + 1 < Q && r >= tab.skip[len + 1] ? 1 : 0);
    send_row(0, b - Q);
    // entries still standing for "baseblock of r": every send round above the top digit
    // and the receive entry of the top digit; one below it the receive entry may be the
    // baseblock of f, which only the search knows
    for (int k = Q - 1; k > top; --k) send_row(k, b);
    recv_row(top, b);
    if (Q > 1 && top > 0 && recv_row.get(top - 1) == kMarkBase) recv_flags |= 1u << (top - 1);
    *send_flags = viol;
    *baseblock_out = b;
    return recv_flags;
}

}  // namespace bcast
