// Instantiations of the chained contraction kernel: token tiles of 160, 192 and 256 rows as CTA pairs.
#include "gemm_tc_kernel.cuh"

namespace dflash {
namespace gemmk {

int gemm_launch_pair(int nt, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int pairs) {
    switch (nt) {
        case 160: return qkn ? launch_pair<160, true>(L, tw, tx, mp, pairs) : launch_pair<160, false>(L, tw, tx, mp, pairs);
        case 192: return qkn ? launch_pair<192, true>(L, tw, tx, mp, pairs) : launch_pair<192, false>(L, tw, tx, mp, pairs);
        default: return qkn ? launch_pair<256, true>(L, tw, tx, mp, pairs) : launch_pair<256, false>(L, tw, tx, mp, pairs);
    }
}

int gemm_pair_capacity(int nt, bool qkn) {
    switch (nt) {
        case 160: return qkn ? pair_capacity<160, true>() : pair_capacity<160, false>();
        case 192: return qkn ? pair_capacity<192, true>() : pair_capacity<192, false>();
        default: return qkn ? pair_capacity<256, true>() : pair_capacity<256, false>();
    }
}

}  // namespace gemmk
}  // namespace dflash
