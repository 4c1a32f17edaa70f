// Instantiations of the warp-MMA kernel for one 16-bit type: include with W4A16_INST_BF (true / false) and
// W4A16_INST_NAME (f16 / bf16) defined.
#include "kernel_tables.h"

namespace w4a16 {
namespace {
template <int SG, bool SYM>
DecodeKernel pick(int mb, bool cluster) {
    constexpr bool BF = W4A16_INST_BF;
    return cluster ? (mb == 2 ? gemm_decode_kernel<2, true, SG, BF, SYM> : gemm_decode_kernel<1, true, SG, BF, SYM>)
                   : (mb == 2 ? gemm_decode_kernel<2, false, SG, BF, SYM> : gemm_decode_kernel<1, false, SG, BF, SYM>);
}
}  // namespace

#define W4A16_CAT2(a, b) a##b
#define W4A16_CAT(a, b) W4A16_CAT2(a, b)

DecodeKernel W4A16_CAT(decode_kernel_, W4A16_INST_NAME)(int mb, bool cluster, int sg, bool sym) {
    if (sym) return sg == 1 ? pick<1, true>(mb, cluster) : sg == 2 ? pick<2, true>(mb, cluster) : pick<4, true>(mb, cluster);
    return sg == 1 ? pick<1, false>(mb, cluster) : sg == 2 ? pick<2, false>(mb, cluster) : pick<4, false>(mb, cluster);
}
int W4A16_CAT(status_take_decode_, W4A16_INST_NAME)() { return status_take_this_unit(); }

}  // namespace w4a16
