// Internal definitions shared by the host packer and the CUDA translation units of libalcs.
// Not part of the public ABI.
#ifndef ALCS_INTERNAL_H_
#define ALCS_INTERNAL_H_

#include <cstddef>
#include <cstdint>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "alcs.h"

namespace alcs {

// Chunk sizes (input channels per pipeline stage) for which a device schedule is prepared at
// upload time.  0 stands for "the whole Cin in one chunk" (used when Cin is small).
constexpr int kNumChunkings = 4;
constexpr int kChunkings[kNumChunkings] = {32, 64, 128, 0};

// Device-resident schedule for one chunk size KC.  Every (block row, chunk) segment of the
// column list is padded to an even number of blocks so that the kernel can fetch column indices
// two at a time with aligned 8-byte loads; a padding block repeats the previous column with
// zero weights.
struct DeviceSchedule {
    int kc = 0;                // channels per chunk (>= 1)
    int nch = 0;               // number of chunks = ceil(cin / kc)
    int nbp = 0;               // padded number of blocks
    int* seg_ptr = nullptr;    // device [R][nch+1], offsets into cols / vals
    int* cols = nullptr;       // device [nbp], chunk-local column index
    float* vals = nullptr;     // device [nbp][g], always fp32 (fp16 weights widened exactly)
};

struct HostSchedule {
    int kc = 0, nch = 0, nbp = 0;
    std::vector<int> seg_ptr, cols;
    std::vector<float> vals;
};

// A resolved launch configuration: which compiled kernel variant, which schedule, how many
// pipeline stages and row groups.
struct Plan {
    int variant = -1;      // index into the table of compiled kernel variants
    int sched = -1;        // index into alcs_packed::sched
    int stages = 0;
    int n_rg = 0;
    int rows_per_rg = 0;
    size_t smem = 0;
    double cost = 0;       // model estimate, seconds
};

struct ShapeKey {
    int n, h, wd;
    unsigned flags;
    bool operator<(const ShapeKey& o) const {
        return std::tie(n, h, wd, flags) < std::tie(o.n, o.h, o.wd, o.flags);
    }
};

}  // namespace alcs

struct alcs_packed {
    int cout = 0, cin = 0, g = 0, rows = 0, nb = 0;
    alcs_dtype dt = ALCS_F32;
    std::vector<int32_t> row_ptr;     // [rows+1]
    std::vector<int32_t> col_idx;     // [nb]
    std::vector<uint8_t> vals;        // [nb*g] elements of dt, raw bytes
    // device side (valid once uploaded)
    int device = -1;
    int* d_row_order = nullptr;       // [rows] block rows by descending kept-block count
    alcs::DeviceSchedule sched[alcs::kNumChunkings];
    std::map<alcs::ShapeKey, alcs_launch_cfg> tuned;   // filled by alcs_spconv1x1_tune
    mutable std::map<alcs::ShapeKey, alcs::Plan> plan_cache;   // resolved plans, by shape
    mutable std::mutex mu;                                      // guards plan_cache
    size_t elt() const { return dt == ALCS_F32 ? 4 : 2; }
};

namespace alcs {

// Host-side helpers implemented in alcs_pack.cpp (no CUDA).
float half_bits_to_float(uint16_t h);
void build_row_order(const alcs_packed& p, std::vector<int>& order);
void build_schedule(const alcs_packed& p, int kc, HostSchedule& out);

}  // namespace alcs

#endif  // ALCS_INTERNAL_H_
