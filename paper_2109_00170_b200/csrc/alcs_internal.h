// Internal definitions shared by the host packer and the CUDA translation units of libalcs.
// Not part of the public ABI.
#ifndef ALCS_INTERNAL_H_
#define ALCS_INTERNAL_H_

#include <cstddef>
#include <array>
#include <cstdint>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "alcs.h"

namespace alcs {

// Chunk sizes (input channels per pipeline stage) the planner considers.  0 stands for "the
// whole Cin in one chunk" (used when Cin is small).
constexpr int kNumChunkings = 6;
constexpr int kChunkings[kNumChunkings] = {16, 32, 64, 96, 128, 0};

// Launch schedule for one (chunk size KC, number of row groups) pair.
//
// Block rows are sorted by descending kept-block count and dealt to the row groups in
// serpentine order, so every row group gets the same number of rows (+-1) and nearly the same
// number of blocks whatever the distribution of row lengths.  rowmap[rg][t] is the block row that
// is local row t of row group rg (-1 = none).
//
// The kept blocks are stored as segments ordered [row group][chunk][local row].  The segment of a
// local row with blocks in a chunk is one "pair record" per two blocks: the chunk-local columns of
// the NEXT pair, then the two g-wide value vectors of this pair (fp32; fp16 weights are widened
// exactly).  An odd block count gets a padding block that repeats the last column with zero
// weights.  slice[rg*nch + k] is where the (row group, chunk) slice starts, so the producer warp
// copies one contiguous range per stage; rowoff[rg][k][t] = {where local row t starts inside that
// slice, the columns of its first pair, its number of pairs}.  Offsets are in 16-byte units.
//
// The balanced flavour (balanced = 1) has the same records, slices and row headers but is built for
// a kernel with nwg consumer warps of rw accumulator sets each.  Row groups hold whole multiples of 4
// rows where possible, every row group has rpg = nwg * rw local rows (unused ones are -1 in the row
// map), and a row group's rows are dealt to the (warp, accumulator set) pairs so that the warps with
// equal index modulo 4 (one scheduler of the SM) get the same number of rows and nearly the same
// number of blocks: the row of (warp w, set s) is local row s*nwg + (s odd ? nwg-1-w : w), the
// kernel's own mapping.  A block row that is far longer than the others of its row group is split
// into parts that take separate (warp, set) pairs (see build_schedule_balanced); for this flavour the
// row-map array is followed by one unit word per local row (unit_word()) and one count of secondary
// units per row group: h_rowmap = [n_rg*rpg rows | n_rg*rpg unit words | n_rg counts].
//
// The tensor-core flavour (mma = 1, fp16 weights, g = 8 or 16) keeps the same slices and row
// headers but stores a segment as "step records" of 16 blocks each: the 16 chunk-local columns
// (uint16), then per 8 output channels the 16x8 weight tile in the register order of the
// m16n8k16 B operand.  The blocks of a segment are ordered so that the 8 columns of each half step
// differ modulo 8 wherever the segment allows it (their shared-memory rows then lie in different
// banks); missing blocks are zero-weight padding.  A row header is {segment start, steps, 0, 0}.
struct Schedule {
    int kc = 0, nch = 0, n_rg = 0, rpg = 0;
    int mma = 0;                   // 1: step records for the tensor-core kernels
    int balanced = 0;              // 1: the balanced flavour (below); then rpg = nwg * rw local rows per row group
    int nwg = 0, rw = 0;           // balanced flavour: consumer warps and accumulator sets per warp it was built for
    int max_x = 0;                 // balanced flavour: most secondary units (parts of split rows) in any row group
    int ros = 0;                   // ints per (row group, chunk) row of rowoff: 4 per local row
    int wcap = 0;                  // longest slice, in 16-byte units
    int n_rec = 0;                 // total length of all slices, in 16-byte units
    // host copies (kept until uploaded)
    std::vector<unsigned char> h_rec;
    std::vector<int> h_slice, h_rowoff, h_rowmap;
    // device copies (valid once uploaded)
    unsigned char* rec = nullptr;
    int* slice = nullptr;
    int* rowoff = nullptr;
    int* rowmap = nullptr;
    bool uploaded = false;
};

// A resolved launch configuration: which compiled kernel variant, which schedule, how many
// pipeline stages.
struct Plan {
    int variant = -1;      // index into the table of compiled kernel variants
    int kc = 0;            // schedule key: channels per chunk ...
    int n_rg = 0;          // ... and number of row groups
    int stages = 0;
    int bulk = 0;          // 0: per-lane cp.async, 1: bulk (TMA) copies of X, 2: per-lane cp.async from rows that are not repacked
    int occ = 1;           // resident thread blocks per SM
    size_t smem = 0;
    double cost = 0;       // model estimate, seconds
    // the small-problem kernel (no staging, reads the canonical format): variant is -1, and
    int gather = 0;        // 1 selects it,
    int gp = 0, gks = 0;   // pixels per lane and warps per thread block (shares of one block row's columns)
};

// Key of the plan cache: the problem shape plus the requested configuration (all zero = automatic).
struct ShapeKey {
    int n, h, wd;
    unsigned flags;
    int c[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    bool operator<(const ShapeKey& o) const {
        if (std::tie(n, h, wd, flags) != std::tie(o.n, o.h, o.wd, o.flags))
            return std::tie(n, h, wd, flags) < std::tie(o.n, o.h, o.wd, o.flags);
        for (int i = 0; i < 12; ++i)
            if (c[i] != o.c[i]) return c[i] < o.c[i];
        return false;
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
    int* d_err = nullptr;             // device error word written by a kernel whose bounded wait ran out
    mutable void* d_xpad = nullptr;   // scratch: X repacked to 16-byte aligned rows (grown on demand)
    // device copy of row_ptr / col_idx / vals for the small-problem kernel (made on first use)
    mutable int32_t* d_row_ptr = nullptr;
    mutable int32_t* d_col_idx = nullptr;
    mutable void* d_vals = nullptr;
    mutable size_t xpad_bytes = 0;
    mutable int max_row_blocks = -1;  // blocks of the longest block row (computed on first use)
    // by (kc, n_rg), built on demand; the tensor-core flavour of a schedule is stored under -kc
    mutable std::map<std::pair<int, int>, alcs::Schedule> sched;
    // schedules of the general k x k convolution, by {row groups, words per channel, words per parity
    // plane, plane pitch, stride, kh, kw, channels per chunk}: the column offsets baked into them depend
    // on the geometry
    mutable std::map<std::array<int, 8>, alcs::Schedule> sched2d;
    mutable std::map<alcs::ShapeKey, alcs_launch_cfg> tuned;   // filled by alcs_spconv1x1_tune, alcs_spconv1x1_set_cfg, alcs_stack_tune
    // the best few plans of the last alcs_spconv1x1_tune per shape, best first: what alcs_stack_tune tries in context
    mutable std::map<alcs::ShapeKey, std::vector<alcs::Plan>> finalists;
    mutable std::map<alcs::ShapeKey, alcs::Plan> plan_cache;   // resolved plans, by shape
    mutable std::mutex mu;                                      // guards plan_cache and sched
    size_t elt() const { return dt == ALCS_F32 ? 4 : 2; }
};

namespace alcs {

// Host-side helpers implemented in alcs_pack.cpp (no CUDA).
float half_bits_to_float(uint16_t h);
float bfloat16_bits_to_float(uint16_t h);
void build_schedule(const alcs_packed& p, int kc, int n_rg, bool with_records, Schedule& out);
void build_schedule_mma(const alcs_packed& p, int kc, int n_rg, bool with_records, Schedule& out);
int pair_record_bytes(int g);                 // bytes of one pair record
int unit_word(int role, int slot, int count);  // see alcs_pack.cpp
int local_row_of(int w, int s, int nw);       // local row of (consumer warp w, accumulator set s), nw consumer warps
void build_schedule_balanced(const alcs_packed& p, int kc, int n_rg, int nwg, int rw, bool with_records, Schedule& out,
                             bool allow_split = true);
// Which flavour of the schedule a kernel takes: 0 = pair records, rows dealt without regard to the
// kernel's shape (the general convolution), 1 = step records of the tensor-core kernels, otherwise
// pair records balanced for (nwg, rw), with or without long block rows split into parts.
constexpr int kMaxBalancedKc = 1 << 19;
inline int balanced_flavour(int nwg, int rw, int split) { return 2 + ((nwg * 16 + rw) << 1 | (split ? 1 : 0)); }
inline int flavour_split(int flavour) { return (flavour - 2) & 1; }
inline int flavour_nwg(int flavour) { return ((flavour - 2) >> 1) / 16; }
inline int flavour_rw(int flavour) { return ((flavour - 2) >> 1) % 16; }
inline std::pair<int, int> sched_key(int kc, int n_rg, int flavour)
{
    if (flavour == 1) return std::make_pair(-kc, n_rg);
    return std::make_pair(flavour >= 2 ? kc + flavour * kMaxBalancedKc : kc, n_rg);
}
// Device-side helpers implemented in alcs_device.cu, for the library's other translation units.
int device_limits(int device, int* sms, int* smem_optin);                 // SM count, opt-in shared memory per block
int schedule_upload(const alcs_packed* w, Schedule* sc, void* cuda_stream); // copy a schedule to w's device (once)
int require_current_device(const alcs_packed* w);                          // ALCS_OK if w is uploaded and its device is current
// bytes of one step record of the tensor-core flavour
constexpr int step_record_bytes(int g) { return 32 + 32 * (g < 8 ? 8 : g); }

}  // namespace alcs

#endif  // ALCS_INTERNAL_H_
