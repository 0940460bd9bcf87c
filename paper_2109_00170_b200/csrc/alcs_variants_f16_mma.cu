// Compiled variants of the tensor-core kernel (fp16 weights and activations, fp32 accumulate).
#include "alcs_mma.cuh"

namespace alcs {

static const KernelVariant kTable[] = {
    //               G  P RW  NW NPW MINB GR
    ALCS_MMA_VARIANT(8, 4, 1, 8, 2, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 2, 8, 2, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 2, 8, 4, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 2, 12, 4, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 1, 12, 4, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 1, 16, 4, 1, 1),
    ALCS_MMA_VARIANT(8, 8, 1, 8, 2, 1, 1),
    ALCS_MMA_VARIANT(8, 8, 1, 8, 4, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 4, 4, 2, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 3, 8, 4, 1, 1),
    ALCS_MMA_VARIANT(8, 4, 1, 8, 2, 2, 1),
    ALCS_MMA_VARIANT(8, 4, 2, 4, 2, 2, 1),
    ALCS_MMA_VARIANT(8, 4, 1, 4, 2, 3, 1),
    ALCS_MMA_VARIANT(8, 4, 2, 6, 2, 2, 1),
    ALCS_MMA_VARIANT(8, 8, 1, 4, 2, 2, 1),
    ALCS_MMA_VARIANT(8, 8, 1, 6, 2, 2, 1),
    ALCS_MMA_VARIANT(8, 4, 1, 16, 4, 1, 2),
    ALCS_MMA_VARIANT(8, 4, 1, 16, 2, 1, 2),
    ALCS_MMA_VARIANT(8, 4, 2, 8, 2, 1, 2),
    ALCS_MMA_VARIANT(8, 4, 2, 8, 4, 1, 2),
    ALCS_MMA_VARIANT(8, 4, 2, 12, 4, 1, 2),
    ALCS_MMA_VARIANT(8, 4, 2, 16, 4, 1, 2),
    ALCS_MMA_VARIANT(8, 4, 4, 8, 4, 1, 2),
    ALCS_MMA_VARIANT(8, 8, 1, 8, 2, 1, 2),
    ALCS_MMA_VARIANT(16, 4, 1, 8, 2, 1, 1),
    ALCS_MMA_VARIANT(16, 4, 1, 16, 4, 1, 2),
    ALCS_MMA_VARIANT(16, 4, 1, 8, 2, 1, 2),
    ALCS_MMA_VARIANT(4, 4, 2, 16, 4, 1, 2),
    ALCS_MMA_VARIANT(16, 4, 1, 8, 4, 1, 1),
    ALCS_MMA_VARIANT(16, 4, 1, 12, 4, 1, 1),
    ALCS_MMA_VARIANT(16, 4, 2, 4, 2, 1, 1),
    ALCS_MMA_VARIANT(16, 8, 1, 4, 2, 1, 1),
    ALCS_MMA_VARIANT(16, 4, 1, 4, 2, 2, 1),
    ALCS_MMA_VARIANT(4, 4, 2, 8, 2, 1, 1),
    ALCS_MMA_VARIANT(4, 4, 2, 12, 4, 1, 1),
    ALCS_MMA_VARIANT(4, 8, 1, 8, 2, 1, 1),
    ALCS_MMA_VARIANT(4, 4, 2, 4, 2, 2, 1),
};

const KernelVariant* variants_f16_mma(int* n)
{
    *n = (int)(sizeof(kTable) / sizeof(kTable[0]));
    return kTable;
}

}  // namespace alcs
