// Long-context build of the persistent decode kernel (8 warps per CTA, both attention modes): head_dim 128,
// GQA group sizes 1..4.  One translation unit per slice of the variants so that they compile in parallel.
#include "megakernel_types.cuh"
#define MK_NS mk_long
#define MK_NW_VALUE MK_NW_LONG
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE

namespace edgefm {

MegaKernel mega_kernel_long_d128_lo(int G) {
    switch (G) {
        case 1: return mk_long::decode_megakernel<128, 1, true>;
        case 2: return mk_long::decode_megakernel<128, 2, true>;
        case 3: return mk_long::decode_megakernel<128, 3, true>;
        case 4: return mk_long::decode_megakernel<128, 4, true>;
    }
    return nullptr;
}

}  // namespace edgefm
