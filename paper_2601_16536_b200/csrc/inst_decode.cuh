// Instantiations of the warp-MMA kernel for one 16-bit type: include with W4A16_INST_BF (true / false) and
// W4A16_INST_NAME (f16 / bf16) defined.
#include "kernel_tables.h"

namespace w4a16 {
namespace {
template <int SG, bool SYM, bool ABOX>
DecodeKernel pick2(int mb, bool cluster) {
    constexpr bool BF = W4A16_INST_BF;
    return cluster ? (mb == 2 ? gemm_decode_kernel<2, true, SG, BF, SYM, ABOX> : gemm_decode_kernel<1, true, SG, BF, SYM, ABOX>)
                   : (mb == 2 ? gemm_decode_kernel<2, false, SG, BF, SYM, ABOX> : gemm_decode_kernel<1, false, SG, BF, SYM, ABOX>);
}
template <int SG, bool SYM>
DecodeKernel pick(int mb, bool cluster, bool a_box) {
    return a_box ? pick2<SG, SYM, true>(mb, cluster) : pick2<SG, SYM, false>(mb, cluster);
}
}  // namespace

#define W4A16_CAT2(a, b) a##b
#define W4A16_CAT(a, b) W4A16_CAT2(a, b)

DecodeKernel W4A16_CAT(decode_kernel_, W4A16_INST_NAME)(int mb, bool cluster, int sg, bool sym, bool a_box) {
    if (sym)
        return sg == 1 ? pick<1, true>(mb, cluster, a_box) : sg == 2 ? pick<2, true>(mb, cluster, a_box) : pick<4, true>(mb, cluster, a_box);
    return sg == 1 ? pick<1, false>(mb, cluster, a_box) : sg == 2 ? pick<2, false>(mb, cluster, a_box) : pick<4, false>(mb, cluster, a_box);
}
int W4A16_CAT(status_take_decode_, W4A16_INST_NAME)() { return status_take_this_unit(); }

}  // namespace w4a16
