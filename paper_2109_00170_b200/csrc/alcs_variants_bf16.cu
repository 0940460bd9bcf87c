// Compiled variants of the bfloat16-input / fp32-accumulate kernel (CUDA cores).  g = 8 is the
// paper's group size for a 16-bit element type on 128-bit SIMD registers (Section 3.2.1).
#include "alcs_kernels.cuh"

namespace alcs {

static const KernelVariant kTable[] = {
    //           XT             dt  G  P RW  NW MINB
    ALCS_VARIANT(__nv_bfloat16, 2, 1, 8, 8, 7, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 2, 8, 4, 7, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 4, 8, 2, 7, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 4, 8, 2, 11, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 8, 8, 1, 7, 2),
    ALCS_VARIANT(__nv_bfloat16, 2, 8, 8, 2, 7, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 8, 8, 1, 15, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 8, 8, 2, 11, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 8, 4, 2, 7, 2),
    ALCS_VARIANT_P(__nv_bfloat16, 2, 8, 8, 1, 14, 1, 2),
    ALCS_VARIANT_P(__nv_bfloat16, 2, 8, 8, 2, 10, 1, 2),
    ALCS_VARIANT(__nv_bfloat16, 2, 16, 4, 1, 7, 2),
    ALCS_VARIANT(__nv_bfloat16, 2, 16, 8, 1, 7, 1),
    ALCS_VARIANT(__nv_bfloat16, 2, 16, 4, 1, 15, 1),
};

const KernelVariant* variants_bf16(int* n)
{
    *n = (int)(sizeof(kTable) / sizeof(kTable[0]));
    return kTable;
}

}  // namespace alcs
