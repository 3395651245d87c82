// Table kernel instantiations for q = 15 .. 20.
#include "table_kernel.cuh"

namespace bcast {

bool launch_table_q_mid(const TableLaunch &l, int q)
{
    switch (q) {
#define BCAST_CASE(N) case N: launch_table_kernel<N>(l); return true;
        BCAST_CASE(15) BCAST_CASE(16) BCAST_CASE(17) BCAST_CASE(18) BCAST_CASE(19) BCAST_CASE(20)
#undef BCAST_CASE
    default: return false;
    }
}

}  // namespace bcast
