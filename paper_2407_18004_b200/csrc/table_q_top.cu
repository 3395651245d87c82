// Table kernel instantiations for q = 26 .. 31.
#include "table_kernel.cuh"

namespace bcast {

bool launch_table_q_top(const TableLaunch &l, int q)
{
    switch (q) {
#define BCAST_CASE(N) case N: launch_table_kernel<N>(l); return true;
        BCAST_CASE(26) BCAST_CASE(27) BCAST_CASE(28) BCAST_CASE(29) BCAST_CASE(30) BCAST_CASE(31)
#undef BCAST_CASE
    default: return false;
    }
}

}  // namespace bcast
