// Block build of the persistent decode kernel: a call carries up to four tokens (the token to decode and three proposed
// continuations to verify; two bf16 pieces per activation), short-context variant, head_dim 64 and 128.
#include "megakernel_types.cuh"
#define MK_NS mk_block4
#define MK_NW_VALUE MK_NW_SHORT
#define MK_M_VALUE 4
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE
#undef MK_M_VALUE

namespace edgefm {

MegaKernel mega_kernel_block4(int head_dim) {
    if (head_dim == 64) return mk_block4::decode_megakernel<64, 1, false>;
    if (head_dim == 128) return mk_block4::decode_megakernel<128, 1, false>;
    return nullptr;
}

}  // namespace edgefm
