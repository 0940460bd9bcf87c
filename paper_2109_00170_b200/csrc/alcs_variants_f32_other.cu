// Compiled variants of the fp32 kernel for group sizes 1 (unstructured CSR), 2, 8 and 16.
#include "alcs_kernels.cuh"

namespace alcs {

static const KernelVariant kTable[] = {
    //           XT   f16  G  P RW  NW MINB
    ALCS_VARIANT(float, 0, 1, 8, 4, 7, 2),
    ALCS_VARIANT(float, 0, 1, 8, 8, 7, 1),
    ALCS_VARIANT(float, 0, 1, 8, 8, 15, 1),
    ALCS_VARIANT(float, 0, 1, 4, 4, 7, 4),
    ALCS_VARIANT(float, 0, 2, 8, 2, 7, 2),
    ALCS_VARIANT(float, 0, 2, 8, 4, 7, 1),
    ALCS_VARIANT(float, 0, 2, 8, 4, 15, 1),
    ALCS_VARIANT(float, 0, 2, 4, 4, 7, 3),
    ALCS_VARIANT(float, 0, 8, 8, 1, 7, 2),
    ALCS_VARIANT(float, 0, 8, 8, 2, 7, 1),
    ALCS_VARIANT(float, 0, 8, 8, 1, 15, 1),
    ALCS_VARIANT(float, 0, 8, 8, 2, 11, 1),
    ALCS_VARIANT(float, 0, 8, 8, 1, 11, 1),
    ALCS_VARIANT(float, 0, 8, 4, 1, 7, 3),
    ALCS_VARIANT(float, 0, 8, 4, 2, 7, 2),
    ALCS_VARIANT(float, 0, 8, 4, 2, 15, 1),
    ALCS_VARIANT(float, 0, 8, 4, 3, 11, 1),
    ALCS_VARIANT(float, 0, 16, 4, 1, 7, 2),
    ALCS_VARIANT(float, 0, 16, 4, 2, 7, 1),
    ALCS_VARIANT(float, 0, 16, 4, 1, 15, 1),
    ALCS_VARIANT(float, 0, 16, 8, 1, 7, 1),
    ALCS_VARIANT(float, 0, 16, 4, 1, 11, 1),
    ALCS_VARIANT(float, 0, 16, 8, 1, 11, 1),
};

const KernelVariant* variants_f32_other(int* n)
{
    *n = (int)(sizeof(kTable) / sizeof(kTable[0]));
    return kTable;
}

}  // namespace alcs
