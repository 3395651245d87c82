// Table kernel instantiations for q = 1 .. 14.
#include "table_kernel.cuh"

namespace bcast {

bool launch_table_q_low(const TableLaunch &l, int q)
{
    switch (q) {
#define BCAST_CASE(N) case N: launch_table_kernel<N>(l); return true;
        BCAST_CASE(1) BCAST_CASE(2) BCAST_CASE(3) BCAST_CASE(4) BCAST_CASE(5) BCAST_CASE(6) BCAST_CASE(7) BCAST_CASE(8) BCAST_CASE(9) BCAST_CASE(10) BCAST_CASE(11) BCAST_CASE(12) BCAST_CASE(13) BCAST_CASE(14)
#undef BCAST_CASE
    default: return false;
    }
}

}  // namespace bcast
