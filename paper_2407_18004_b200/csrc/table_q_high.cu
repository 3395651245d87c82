// Table kernel instantiations for q = 21 .. 25.
#include "table_kernel.cuh"

namespace bcast {

bool launch_table_q_high(const TableLaunch &l, int q)
{
    switch (q) {
#define BCAST_CASE(N) case N: launch_table_kernel<N>(l); return true;
        BCAST_CASE(21) BCAST_CASE(22) BCAST_CASE(23) BCAST_CASE(24) BCAST_CASE(25)
#undef BCAST_CASE
    default: return false;
    }
}

}  // namespace bcast
