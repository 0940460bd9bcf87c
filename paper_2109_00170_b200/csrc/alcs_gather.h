// Launcher of the small-problem (direct gather) kernel of the sparse pointwise convolution.
// Internal to libalcs.
#ifndef ALCS_GATHER_H_
#define ALCS_GATHER_H_

#include <cuda_runtime.h>

namespace alcs {

struct GatherArgs {
    const float* x;           // [n][cin][hw]
    float* y;                 // [n][cout][hw]
    const float* bias;        // [cout] or nullptr
    const int* row_ptr;       // the canonical storage format, on the device
    const int* col_idx;
    const float* vals;
    int rows, cin, cout, hw, n;
    int tiles;                // pixel tiles of 32 * P per image
    int relu;
    int vec;                  // 1: rows of x are 16-byte aligned multiples of 4 pixels
    int stage_blocks;         // block rows of at most this many blocks are copied into shared memory before
                              // the kernel waits for its predecessor (0: none; see gather_stage_blocks)
};

// g in {1,2,4,8,16}, p = pixels per lane in {2,4,8}, ks = warps per thread block (1..16) that share one
// block row's columns.
bool gather_config_ok(int g, int p, int ks, bool vec);
cudaError_t launch_gather(int g, int p, int ks, const GatherArgs& a, cudaStream_t st);
// The value of GatherArgs::stage_blocks for a matrix whose longest block row has max_row_blocks blocks: that
// length if such a row fits in 48 KB of shared memory, else 0.
int gather_stage_blocks(int g, int max_row_blocks);

}  // namespace alcs

#endif  // ALCS_GATHER_H_
