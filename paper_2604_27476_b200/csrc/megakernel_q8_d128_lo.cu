// Long-context build of the persistent decode kernel for the compressed KV cache (8-bit codes and a scale per cached
// row): head_dim 128, GQA group sizes 1..4.  One translation unit per slice of the variants so that they compile in parallel.
#include "megakernel_types.cuh"
#define MK_NS mk_long
#define MK_NW_VALUE MK_NW_LONG
#include "megakernel.cuh"
#undef MK_NS
#undef MK_NW_VALUE

namespace edgefm {

MegaKernel mega_kernel_q8_d128_lo(int G) {
    switch (G) {
        case 1: return mk_long::decode_megakernel<128, 1, true, true>;
        case 2: return mk_long::decode_megakernel<128, 2, true, true>;
        case 3: return mk_long::decode_megakernel<128, 3, true, true>;
        case 4: return mk_long::decode_megakernel<128, 4, true, true>;
    }
    return nullptr;
}

}  // namespace edgefm
