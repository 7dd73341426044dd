// Long-context build of the persistent decode kernel for the compressed KV cache (8-bit codes and a scale per cached
// row): head_dim 128, GQA group sizes 5..8.  One translation unit per slice of the variants so that they compile in parallel.
#include "megakernel_types.cuh"
#define MK_NS mk_long
#define MK_NW_VALUE MK_NW_LONG
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE

namespace edgefm {

MegaKernel mega_kernel_q8_d128_hi(int G) {
    switch (G) {
        case 5: return mk_long::decode_megakernel<128, 5, true, true>;
        case 6: return mk_long::decode_megakernel<128, 6, true, true>;
        case 7: return mk_long::decode_megakernel<128, 7, true, true>;
        case 8: return mk_long::decode_megakernel<128, 8, true, true>;
    }
    return nullptr;
}

}  // namespace edgefm
