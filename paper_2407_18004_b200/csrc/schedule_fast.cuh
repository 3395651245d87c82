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
//    digit above k, minus q); with no digit above k it is the baseblock of f, or
//    k itself when f is the root.
//  * Digit k clear: subtracting skip[k] borrows from the lowest set digit j above
//    k.  f's walk equals r's above j, is in the lower part at j, and below j it
//    is in the upper part at every level down to k+1 exactly when
//        X = r'_j - skip[k] - (skip[k+1] + ... + skip[j-1])  >= 0,
//    r'_j being r's virtual index entering level j; X is then f's virtual index
//    entering level k and e_j' - (same sum) its bound, which is all round k's
//    rule needs.  Prefix sums of the skips make this O(1).
//  * Whenever the rule reports a violation for (f, k), or X < 0, or the value
//    would be a baseblock this pass cannot know, the entry is flagged and the
//    caller computes it with the search of Algorithms 4 and 5.
//
// Q is a template parameter so that the level loop unrolls completely: skips and
// prefix sums become constant-bank operands and row offsets immediates.
#pragma once
#include <stdint.h>

namespace bcast {

struct LevelTables {
    uint32_t skip[33];      // skip[0..q]
    uint32_t below[34];     // below[l] = skip[0] + ... + skip[l-1]
};

constexpr int kMarkBase = 100;      // stands for "the baseblock of r" until it is known

// Rows of virtual rank r >= 1.  recv_row/send_row: (k, value) writers that can also
// read back an entry.  Returns the rounds whose receive entry must come from the
// search; *send_flags receives the rounds whose send entry must (Algorithm 6's
// violations).
template <int Q, class Row>
__device__ __forceinline__ uint32_t closed_form_rows(const LevelTables &tab, uint32_t p, uint32_t r,
                                                     Row recv_row, Row send_row, uint32_t *send_flags)
{
    uint32_t rp = r;                 // Algorithm 6: virtual processor index r'
    uint32_t e = p;                  //              bound on the virtual range
    int c = kMarkBase;               //              block the lower part sends
    // state of r's walk entering the lowest upper level j seen so far (j = q at first)
    uint32_t rpJ = p + r;            // r' entering level j
    uint32_t eJ = p;                 // min(e entering level j, skip[j])
    int cJ = kMarkBase;              // c entering level j
    uint32_t belowJ = tab.below[Q];  // skip[0] + ... + skip[j-1]
    int j = Q;
    int top = -1;                    // highest set digit of r
    uint32_t recv_flags = 0, viol = 0;

#pragma unroll
    for (int k = Q - 1; k >= 0; --k) {
        const uint32_t sk = tab.skip[k];
        const uint32_t sk_below = k > 0 ? tab.skip[k - 1] : 0u;
        if (rp >= sk) {                                              // upper part: digit k set
            const int rv = c != kMarkBase ? c : (rp == sk ? k : kMarkBase);
            recv_row(k, rv);
            if (k > 0) {
                if (k > 1 && rp == sk && e - sk >= sk_below && rp + sk > e) viol |= 1u << k;
                send_row(k, k - Q);
            }
            if (c == kMarkBase) top = k;
            rpJ = rp; eJ = min(e, sk); cJ = c; belowJ = tab.below[k]; j = k;
            c = k - Q;
            rp -= sk;
            e -= sk;
        } else {                                                     // lower part: digit k clear
            if (k > 0) {
                if (!(rp + sk < e || e < sk_below || (k == 1 && rp == 0u))) viol |= 1u << k;
                send_row(k, c);
            }
            // round-k rule of Algorithm 6 for f = R - skip[k]
            const uint32_t sum = belowJ - tab.below[k + 1];          // skip[k+1..j-1]
            const uint32_t need = sk + sum;
            const bool all_upper = rpJ >= need;
            const uint32_t X = rpJ - need;
            const uint32_t eB = eJ - sum;
            const int cB = j > k + 1 ? k + 1 - Q : cJ;
            bool bad;
            int rv;
            if (X >= sk) {
                rv = k - Q;
                bad = k > 1 && X == sk && eB - sk >= sk_below && X + sk > eB;
            } else {
                rv = cB;
                bad = cB == kMarkBase ||
                      (k > 0 && !(X + sk < eB || eB < sk_below || (k == 1 && X == 0u)));
            }
            if (!all_upper || bad) recv_flags |= 1u << k;
            recv_row(k, rv);
            e = min(e, sk);
        }
    }
    // j is now the lowest set digit of r: its baseblock
    const int b = j;
    send_row(0, b - Q);
    // entries that stand for "baseblock of r": the send rounds above r's top digit and
    // possibly the receive entry of the top digit itself
    for (int k = Q - 1; k > top; --k) send_row(k, b);
    if (recv_row.get(top) == kMarkBase) recv_row(top, b);
    *send_flags = viol;
    return recv_flags;
}

}  // namespace bcast
