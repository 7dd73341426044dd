// Block build of the persistent decode kernel: a call carries up to two tokens (the token to decode and one proposed
// continuation to verify), short-context variant, head_dim 64 and 128.
#include "megakernel_types.cuh"
#define MK_NS mk_block2
#define MK_NW_VALUE MK_NW_SHORT
#define MK_M_VALUE 2
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE
#undef MK_M_VALUE

namespace edgefm {

MegaKernel mega_kernel_block2(int head_dim) {
    if (head_dim == 64) return mk_block2::decode_megakernel<64, 1, false>;
    if (head_dim == 128) return mk_block2::decode_megakernel<128, 1, false>;
    return nullptr;
}

}  // namespace edgefm
