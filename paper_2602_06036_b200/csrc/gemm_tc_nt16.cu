// Instantiations of the chained contraction kernel: token tiles of 16 rows.
#include "gemm_tc_kernel.cuh"

namespace dflash {
namespace gemmk {

int gemm_launch_16(int slabs, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid) {
    if (slabs == 2) return qkn ? launch_nt<16, 2, true>(L, tw, tx, mp, grid) : launch_nt<16, 2, false>(L, tw, tx, mp, grid);
    return qkn ? launch_nt<16, 1, true>(L, tw, tx, mp, grid) : launch_nt<16, 1, false>(L, tw, tx, mp, grid);
}

}  // namespace gemmk
}  // namespace dflash
