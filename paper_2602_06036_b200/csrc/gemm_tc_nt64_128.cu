// Instantiations of the chained contraction kernel: token tiles of 64 and 128 rows.
#include "gemm_tc_kernel.cuh"

namespace dflash {
namespace gemmk {

int gemm_launch_64_128(int nt, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid) {
    if (nt == 64) return qkn ? launch_nt<64, 1, true>(L, tw, tx, mp, grid) : launch_nt<64, 1, false>(L, tw, tx, mp, grid);
    return qkn ? launch_nt<128, 1, true>(L, tw, tx, mp, grid) : launch_nt<128, 1, false>(L, tw, tx, mp, grid);
}

}  // namespace gemmk
}  // namespace dflash
