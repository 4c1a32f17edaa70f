// Instantiations of the tcgen05 tile kernel for one 16-bit type and group size: include with W4A16_INST_BF
// (true / false), W4A16_INST_SG (1 / 2 / 4) and W4A16_INST_NAME (f16_sg1 ...) defined.
#include "kernel_tables.h"

namespace w4a16 {
namespace {
template <bool SYM, bool EPI>
TileKernel pick(int mt_index) {
    constexpr bool BF = W4A16_INST_BF;
    constexpr int SG = W4A16_INST_SG;
    return mt_index == 0 ? gemm_tile_kernel<16, SG, BF, SYM, EPI> : mt_index == 1 ? gemm_tile_kernel<32, SG, BF, SYM, EPI>
         : mt_index == 2 ? gemm_tile_kernel<64, SG, BF, SYM, EPI> : mt_index == 3 ? gemm_tile_kernel<128, SG, BF, SYM, EPI>
                                                                                   : gemm_tile_kernel<256, SG, BF, SYM, EPI>;
}
}  // namespace

#define W4A16_CAT2(a, b) a##b
#define W4A16_CAT(a, b) W4A16_CAT2(a, b)

TileKernel W4A16_CAT(tile_kernel_, W4A16_INST_NAME)(int mt_index, bool sym, bool epi) {
    if (sym) return epi ? pick<true, true>(mt_index) : pick<true, false>(mt_index);
    return epi ? pick<false, true>(mt_index) : pick<false, false>(mt_index);
}
int W4A16_CAT(status_take_tile_, W4A16_INST_NAME)() { return status_take_this_unit(); }

}  // namespace w4a16
