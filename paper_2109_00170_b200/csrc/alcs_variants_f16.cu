// Compiled variants of the fp16-input / fp32-accumulate kernel.
#include "alcs_kernels.cuh"

namespace alcs {

static const KernelVariant kTable[] = {
    //           XT   f16  G  P RW  NW MINB
    ALCS_VARIANT(__half, 1, 1, 8, 8, 7, 1),
    ALCS_VARIANT(__half, 1, 2, 8, 4, 7, 1),
    ALCS_VARIANT(__half, 1, 4, 8, 2, 7, 1),
    ALCS_VARIANT(__half, 1, 4, 8, 2, 11, 1),
    ALCS_VARIANT(__half, 1, 4, 4, 2, 7, 2),
    ALCS_VARIANT(__half, 1, 8, 8, 1, 7, 2),
    ALCS_VARIANT(__half, 1, 8, 8, 2, 7, 1),
    ALCS_VARIANT(__half, 1, 8, 8, 1, 15, 1),
    ALCS_VARIANT(__half, 1, 8, 8, 2, 11, 1),
    ALCS_VARIANT(__half, 1, 8, 8, 1, 11, 1),
    ALCS_VARIANT(__half, 1, 8, 4, 2, 7, 2),
    ALCS_VARIANT(__half, 1, 8, 4, 1, 7, 3),
    ALCS_VARIANT(__half, 1, 16, 4, 1, 7, 2),
    ALCS_VARIANT(__half, 1, 16, 8, 1, 7, 1),
    ALCS_VARIANT(__half, 1, 16, 4, 1, 15, 1),
    ALCS_VARIANT(__half, 1, 16, 8, 1, 11, 1),
};

const KernelVariant* variants_f16(int* n)
{
    *n = (int)(sizeof(kTable) / sizeof(kTable[0]));
    return kTable;
}

}  // namespace alcs
