// Long-context build of the persistent decode kernel (8 warps per CTA, both attention modes): head_dim 64,
// GQA group sizes 5..8.  One translation unit per slice of the variants so that they compile in parallel.
#include "megakernel_types.cuh"
#define MK_NS mk_long
#define MK_NW_VALUE MK_NW_LONG
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE

namespace edgefm {

MegaKernel mega_kernel_long_d64_hi(int G) {
    switch (G) {
        case 5: return mk_long::decode_megakernel<64, 5, true>;
        case 6: return mk_long::decode_megakernel<64, 6, true>;
        case 7: return mk_long::decode_megakernel<64, 7, true>;
        case 8: return mk_long::decode_megakernel<64, 8, true>;
    }
    return nullptr;
}

}  // namespace edgefm
