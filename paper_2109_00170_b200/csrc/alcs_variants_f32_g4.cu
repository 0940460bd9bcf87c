// Compiled variants of the fp32, g = 4 kernel (the paper's group size for 32-bit weights on
// 128-bit SIMD registers, Section 4.1).
#include "alcs_kernels.cuh"

namespace alcs {

static const KernelVariant kTable[] = {
    //             XT   f16  G  P RW  NW MINB NPW
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 3, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 4, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 4, 6, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 7, 2, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 7, 2, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 6, 2, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 11, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 11, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 3, 11, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 10, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 3, 10, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 15, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 15, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 14, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 14, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 13, 1, 3),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 13, 1, 3),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 12, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 12, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 2, 12, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 3, 8, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 8, 3, 8, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 16, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 16, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 19, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 8, 1, 18, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 2, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 6, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 7, 2, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 2, 7, 2, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 6, 2, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 2, 11, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 11, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 6, 11, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 10, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 6, 10, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 2, 15, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 15, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 14, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 2, 23, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 12, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 12, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 6, 8, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 4, 2, 16, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 4, 3, 16, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 4, 4, 16, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 8, 6, 1, 2),
    ALCS_VARIANT_P(float, 0, 4, 4, 8, 8, 1, 4),
    ALCS_VARIANT_P(float, 0, 4, 16, 1, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 16, 1, 11, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 16, 2, 7, 1, 1),
    ALCS_VARIANT_P(float, 0, 4, 16, 1, 10, 1, 2),
    // the same kernels for schedules with block rows split into parts (skewed row lengths)
    ALCS_VARIANT_SPLIT(float, 0, 4, 8, 2, 12, 1, 4),
    ALCS_VARIANT_SPLIT(float, 0, 4, 8, 2, 12, 1, 2),
    ALCS_VARIANT_SPLIT(float, 0, 4, 8, 2, 14, 1, 2),
    ALCS_VARIANT_SPLIT(float, 0, 4, 8, 1, 16, 1, 4),
    ALCS_VARIANT_SPLIT(float, 0, 4, 8, 3, 8, 1, 4),
    ALCS_VARIANT_SPLIT(float, 0, 4, 4, 3, 16, 1, 4),
    ALCS_VARIANT_SPLIT(float, 0, 4, 4, 4, 12, 1, 4),
    ALCS_VARIANT_SPLIT(float, 0, 4, 4, 2, 16, 1, 4),
};

const KernelVariant* variants_f32_g4(int* n)
{
    *n = (int)(sizeof(kTable) / sizeof(kTable[0]));
    return kTable;
}

}  // namespace alcs
