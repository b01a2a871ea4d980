// Instantiations of the chained contraction kernel: token tiles of 160, 192 and 256 rows, one CTA per MMA.
#include "gemm_tc_kernel.cuh"

namespace dflash {
namespace gemmk {

int gemm_launch_160_256(int nt, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid) {
    switch (nt) {
        case 160: return qkn ? launch_nt<160, 1, true>(L, tw, tx, mp, grid) : launch_nt<160, 1, false>(L, tw, tx, mp, grid);
        case 192: return qkn ? launch_nt<192, 1, true>(L, tw, tx, mp, grid) : launch_nt<192, 1, false>(L, tw, tx, mp, grid);
        default: return qkn ? launch_nt<256, 1, true>(L, tw, tx, mp, grid) : launch_nt<256, 1, false>(L, tw, tx, mp, grid);
    }
}

}  // namespace gemmk
}  // namespace dflash
