// Device code of the SIMD-structured sparse pointwise convolution for sm_100a.
//
// Work decomposition (see the paper's Section 3.2.2, "Efficient multiplication computation", for
// the loop this re-creates: zero the accumulators, loop over a group's kept columns, multiply the
// column's g weights with the input vector addressed by the column offset, accumulate):
//
//   work item    = one tile of T = 32*P consecutive pixels (pixels of all images flattened,
//                  q = n*HW + p) x one "row group" (a balanced subset of the block rows)
//   thread block = persistent: walks items blockIdx.x, blockIdx.x + gridDim.x, ...
//   consumer warp= RW block rows at a time, all T pixels of the tile
//   lane         = P pixels of each of those rows: G*P fp32 accumulators per row in registers
//   producer warps= one or more extra warps that only move data
//
// The input channels are walked in chunks of KC channels.  For each (item, chunk) the producer
// warp copies, with cp.async, the X tile ([KC][T] elements) and the row group's slice of the
// packed weights for that chunk (one contiguous range of "pair records": two column indices and
// their two g-wide value vectors) into one stage of a shared-memory ring that runs on across
// items, so the loads of the next tile overlap the arithmetic and the stores of the current
// one.  Stages are handed over through mbarriers: "full" is completed by the producer lanes'
// cp.async completion, "empty" by one arrival per consumer warp, so consumer warps never wait
// for each other, only for data.  In the hot loop everything is a shared-memory load: records
// are warp-uniform broadcasts, X values are 128-bit conflict-free loads, and every X word feeds
// G FMAs.
//
// Every mbarrier wait is bounded: after kWaitLimit polls the warp records an error code in
// ConvArgs::err and leaves the kernel (the producer first waits for its own copies).
#ifndef ALCS_KERNELS_CUH_
#define ALCS_KERNELS_CUH_

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <type_traits>

namespace alcs {

constexpr int kMaxStages = 8;
constexpr int kWaitLimit = 1 << 21;     // polls of mbarrier.try_wait before giving up (about a second)
constexpr int kErrFullWait = 1;         // a consumer gave up waiting for data
constexpr int kErrEmptyWait = 2;        // the producer gave up waiting for a free stage

// Bytes of one pair record: a header with the two column indices of the NEXT pair of the segment
// (padded to 16 bytes unless G == 1, where the two values share the header's 16 bytes) followed
// by the 2*G fp32 values of this pair.  A segment starts with a 16-byte lead entry that holds the
// column indices of its first pair.
__host__ __device__ constexpr int record_bytes(int g) { return g == 1 ? 16 : 16 + 8 * g; }

struct ConvArgs {
    const void* x;            // [n][cin][hw] of XT
    void* y;                  // [n][cout][hw] of XT, or float if y_f32
    const float* bias;        // [cout] or nullptr
    const void* res;          // residual, same shape and element type as y, or nullptr: y = act(acc + bias + res)
    const unsigned char* rec; // segments of pair records, ordered [row group][chunk][local row]
    const int* slice;         // [n_rg*nch + 1] start of each (row group, chunk) slice, in 16-byte units
    const int* rowoff;        // [n_rg][nch][rpg] int4 per local row: {segment start inside the slice (16-byte units), c0, c1, pairs}
    const int* rowmap;        // [n_rg][rpg] block row of each local row, -1 = none
    const int* unit;          // [n_rg][rpg] unit word of each local row (role | slot << 4 | count << 16), or nullptr when
                              // no block row of the schedule is split into parts
    const int* rgx;           // [n_rg] secondary units per row group (0: no hand-over in that row group)
    int off_xch;              // shared memory: hand-over area [mbarrier, 16 bytes | 2 x xch_slots tiles of G*P*32 floats]
    int xch_slots;
    int* err;                 // device error word (0 = ok)
    int rows, cin, cout;
    int hw;                   // pixels per image in X (padded up when X was repacked to aligned rows)
    int hwy;                  // pixels per image in Y (the real h*w, <= hw)
    int q_total;              // n * hw
    int n_tiles, n_rg, rpg;   // pixel tiles, row groups, local rows per row group (padded)
    int kc, nch, stages;
    int relu;
    int y_f32;                // only meaningful for XT = __half
    int ld_bytes;             // bytes per X staging copy: 16, 8, 4 or 2
    int bulk;                 // 1: the producer uses bulk (TMA) copies; needs ld_bytes == 16.  2: the same, and x is a
                              // tile-major copy of the input: [pixel tile][channel][32*P pixels (+ row padding)], so
                              // that the channel rows of a chunk are one contiguous run
    int ros;                  // ints of rowoff per (row group, chunk): 4 per header
    int st_vec;               // 1 if vector stores are allowed
    int st_grp;               // 1 if the pixels of one vector store of a lane always lie in one image; 2 (tensor-core
                              // kernel, 16-bit output): store single elements, consecutive lanes on consecutive pixels
    // shared-memory layout (bytes): [mbarriers | stage 0 | stage 1 | ...]
    int off_rec, off_rowoff, stage_bytes;
};

// ---- small PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_8(uint32_t dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.wait_all;\n" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("{\n .reg .b64 t;\n mbarrier.arrive.shared::cta.b64 t, [%0];\n}\n" ::"r"(bar) : "memory");
}
// Arrive on `bar` once all cp.async copies this thread has issued so far have landed.
__device__ __forceinline__ void mbar_arrive_on_copies(uint32_t bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}
// One arrival that also announces `bytes` of bulk-copy traffic still to land on `bar`.
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("{\n .reg .b64 t;\n mbarrier.arrive.expect_tx.shared::cta.b64 t, [%0], %1;\n}\n" ::"r"(bar), "r"(bytes)
                 : "memory");
}
// Bulk asynchronous copy global -> shared memory (TMA, untiled): 16-byte aligned addresses, size a
// multiple of 16; its bytes are counted down on `bar` when they have landed.  No multicast.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute
// may start while the previous kernel on the stream is still draining.  grid_dep_wait() blocks until
// that previous kernel has completed and its writes are visible; everything that touches X, Y or the
// repack scratch comes after it, so only set-up work (barrier init, the first weight copies)
// overlaps the predecessor's tail.  grid_dep_launch() lets the NEXT kernel start its own set-up.
// Both are no-ops for an ordinary launch.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// Bounded wait for the phase with the given parity to complete.  Each poll lets the hardware
// suspend the warp until the phase completes or a time limit passes, so a waiting warp takes few
// issue slots from the warps that compute; the warp is not put to sleep between polls, because a
// sleeping warp notices the hand-over of a pipeline stage up to a sleep period late, and with two
// or three stages that delay sits on the critical path of every chunk.  Only a wait that has already
// lasted thousands of polls backs off with nanosleep.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (int it = 0; it < kWaitLimit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
            " selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(done)
            : "r"(bar), "r"(parity), "r"(1000u)
            : "memory");
        if (done) return true;
        if (it > 4096) __nanosleep(128);
    }
    return false;
}

// Load VG consecutive X elements from shared memory and widen them to fp32.
template <typename XT, int VG>
struct XVec;
template <>
struct XVec<float, 4> {
    static __device__ __forceinline__ void load(const unsigned char* p, float (&x)[4])
    {
        const float4 v = *reinterpret_cast<const float4*>(p);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
};
template <>
struct XVec<__half, 8> {
    static __device__ __forceinline__ void load(const unsigned char* p, float (&x)[8])
    {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
};
template <>
struct XVec<__half, 4> {
    static __device__ __forceinline__ void load(const unsigned char* p, float (&x)[4])
    {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float2 f = __half22float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
};

template <>
struct XVec<__nv_bfloat16, 8> {
    static __device__ __forceinline__ void load(const unsigned char* p, float (&x)[8])
    {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
};
template <>
struct XVec<__nv_bfloat16, 4> {
    static __device__ __forceinline__ void load(const unsigned char* p, float (&x)[4])
    {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
};

// The P pixels a lane owns of one staged channel row, as P/2 adjacent pairs: P/VG vector loads,
// 32*VG elements apart.
template <typename XT, int P>
__device__ __forceinline__ void load_x(const unsigned char* p, float2 (&x)[P / 2])
{
    constexpr int SZ = (int)sizeof(XT);
    constexpr int VG = (P * SZ >= 16) ? 16 / SZ : P;
#pragma unroll
    for (int gi = 0; gi < P / VG; ++gi) {
        float v[VG];
        XVec<XT, VG>::load(p + gi * (32 * VG * SZ), v);
#pragma unroll
        for (int t = 0; t < VG / 2; ++t) x[gi * (VG / 2) + t] = make_float2(v[2 * t], v[2 * t + 1]);
    }
}

// One pair record from shared memory (same address in every lane: broadcasts).
template <int G>
__device__ __forceinline__ void load_record(const unsigned char* p, int& c0, int& c1, float (&w0)[G],
                                            float (&w1)[G])
{
    const int4 h = *reinterpret_cast<const int4*>(p);
    c0 = h.x;
    c1 = h.y;
    if constexpr (G == 1) {
        w0[0] = __int_as_float(h.z);
        w1[0] = __int_as_float(h.w);
    } else if constexpr (G == 2) {
        const float4 v = *reinterpret_cast<const float4*>(p + 16);
        w0[0] = v.x; w0[1] = v.y; w1[0] = v.z; w1[1] = v.w;
    } else {
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 v = *reinterpret_cast<const float4*>(p + 16 + 16 * i);
            w0[4 * i] = v.x; w0[4 * i + 1] = v.y; w0[4 * i + 2] = v.z; w0[4 * i + 3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 v = *reinterpret_cast<const float4*>(p + 16 + 4 * G + 16 * i);
            w1[4 * i] = v.x; w1[4 * i + 1] = v.y; w1[4 * i + 2] = v.z; w1[4 * i + 3] = v.w;
        }
    }
}

// G (>= 4) weights of one block from shared memory (warp-uniform address).
template <int G>
__device__ __forceinline__ void load_w(const unsigned char* p, float (&w)[G])
{
#pragma unroll
    for (int i = 0; i < G / 4; ++i) {
        const float4 v = *reinterpret_cast<const float4*>(p + 16 * i);
        w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
    }
}

// acc[j][t] += w[j] * x[t]: the G x P outer-product update of one block, two pixels per
// instruction with the packed fp32 FMA of sm_100 (each half is an IEEE fused multiply-add, so
// the result equals the scalar fmaf bit for bit).  Fewer issue slots per FMA leave room for the
// shared-memory loads and the loop bookkeeping.
template <int G, int P>
__device__ __forceinline__ void fma_block(float2 (&acc)[G][P / 2], const float (&w)[G], const float2 (&x)[P / 2])
{
#pragma unroll
    for (int j = 0; j < G; ++j) {
        const float2 w2 = make_float2(w[j], w[j]);
#pragma unroll
        for (int t = 0; t < P / 2; ++t) acc[j][t] = __ffma2_rn(w2, x[t], acc[j][t]);
    }
}

// Multiply-accumulate one (block row, chunk) segment of `npairs` pair records, starting at rp in
// shared memory, into the lane's G x P accumulators.  xs points at this lane's first pixel vector
// of the staged X tile; (ca0, ca1) are the columns of the first pair.
template <typename XT, int G, int P, bool DEEP>
__device__ __forceinline__ void consume_segment(float2 (&acc)[G][P / 2], const unsigned char* xs,
                                                const unsigned char* rp, int npairs, int ca0, int ca1)
{
    constexpr int ROWB = 32 * P * (int)sizeof(XT);
    constexpr int REC = record_bytes(G);
    // A segment is one record per pair, holding the columns of the NEXT pair and the weights of
    // this one; the columns of pair 0 (ca0, ca1) come with the segment's header.  So the loads
    // issued while pair i is multiplied (record i+1, X vectors of pair i+1) depend only on data
    // that arrived while pair i-1 was multiplied.  Two register sets (A, B) alternate; nothing is
    // copied between them.
    const unsigned char* re = rp + npairs * REC;
    int cb0 = 0, cb1 = 0;
    if constexpr (G <= 4 && DEEP) {
        float wA0[G], wA1[G], wB0[G], wB1[G];
        float2 xA0[P / 2], xA1[P / 2], xB0[P / 2], xB1[P / 2];
        load_record<G>(rp, cb0, cb1, wA0, wA1);
        load_x<XT, P>(xs + ca0 * ROWB, xA0);
        load_x<XT, P>(xs + ca1 * ROWB, xA1);
        while (true) {
            const bool moreB = rp + REC < re;
            if (moreB) {
                load_record<G>(rp + REC, ca0, ca1, wB0, wB1);
                load_x<XT, P>(xs + cb0 * ROWB, xB0);
                load_x<XT, P>(xs + cb1 * ROWB, xB1);
            }
            fma_block<G, P>(acc, wA0, xA0);
            fma_block<G, P>(acc, wA1, xA1);
            if (!moreB) break;
            const bool moreA = rp + 2 * REC < re;
            if (moreA) {
                load_record<G>(rp + 2 * REC, cb0, cb1, wA0, wA1);
                load_x<XT, P>(xs + ca0 * ROWB, xA0);
                load_x<XT, P>(xs + ca1 * ROWB, xA1);
            }
            fma_block<G, P>(acc, wB0, xB0);
            fma_block<G, P>(acc, wB1, xB1);
            if (!moreA) break;
            rp += 2 * REC;
        }
    } else if constexpr (G <= 4) {
        // Register-lean flavour for thread blocks with many warps: only the records are fetched
        // ahead (two alternating weight sets); the X vectors of a pair are loaded when the
        // previous pair's FMAs have been issued, and other warps cover that latency.
        float wA0[G], wA1[G], wB0[G], wB1[G];
        float2 x0[P / 2], x1[P / 2];
        load_record<G>(rp, cb0, cb1, wA0, wA1);
        load_x<XT, P>(xs + ca0 * ROWB, x0);
        load_x<XT, P>(xs + ca1 * ROWB, x1);
        while (true) {
            const bool moreB = rp + REC < re;
            if (moreB) load_record<G>(rp + REC, ca0, ca1, wB0, wB1);
            fma_block<G, P>(acc, wA0, x0);
            fma_block<G, P>(acc, wA1, x1);
            if (!moreB) break;
            load_x<XT, P>(xs + cb0 * ROWB, x0);
            load_x<XT, P>(xs + cb1 * ROWB, x1);
            const bool moreA = rp + 2 * REC < re;
            if (moreA) load_record<G>(rp + 2 * REC, cb0, cb1, wA0, wA1);
            fma_block<G, P>(acc, wB0, x0);
            fma_block<G, P>(acc, wB1, x1);
            if (!moreA) break;
            load_x<XT, P>(xs + ca0 * ROWB, x0);
            load_x<XT, P>(xs + ca1 * ROWB, x1);
            rp += 2 * REC;
        }
    } else {
        // Wide groups: every X word already feeds 8 or 16 FMAs and the accumulators
        // fill most of the register file, so nothing but the next pair's columns is
        // fetched ahead; the weights of each block are loaded just before its FMAs.
        while (true) {
            float2 x0[P / 2], x1[P / 2];
            float w[G];
            load_x<XT, P>(xs + ca0 * ROWB, x0);
            load_x<XT, P>(xs + ca1 * ROWB, x1);
            const int2 nx = *reinterpret_cast<const int2*>(rp);
            load_w<G>(rp + 16, w);
            fma_block<G, P>(acc, w, x0);
            load_w<G>(rp + 16 + 4 * G, w);
            fma_block<G, P>(acc, w, x1);
            if (rp + REC >= re) break;
            ca0 = nx.x;
            ca1 = nx.y;
            rp += REC;
        }
    }
}

template <typename YT, int VG>
__device__ __forceinline__ void store_vec(YT* p, const float (&v)[VG])
{
    if constexpr (sizeof(YT) == 4) {
#pragma unroll
        for (int i = 0; i < VG / 4; ++i)
            reinterpret_cast<float4*>(p)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else if constexpr (std::is_same<YT, __half>::value) {
        __half2 h[VG / 2];
#pragma unroll
        for (int i = 0; i < VG / 2; ++i) h[i] = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
        if constexpr (VG == 8)
            *reinterpret_cast<uint4*>(p) = *reinterpret_cast<const uint4*>(h);
        else
            *reinterpret_cast<uint2*>(p) = *reinterpret_cast<const uint2*>(h);
    } else {
        __nv_bfloat162 h[VG / 2];
#pragma unroll
        for (int i = 0; i < VG / 2; ++i) h[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        if constexpr (VG == 8)
            *reinterpret_cast<uint4*>(p) = *reinterpret_cast<const uint4*>(h);
        else
            *reinterpret_cast<uint2*>(p) = *reinterpret_cast<const uint2*>(h);
    }
}

template <typename YT>
__device__ __forceinline__ void store_one(YT* p, float v)
{
    if constexpr (sizeof(YT) == 4)
        *p = v;
    else if constexpr (std::is_same<YT, __half>::value)
        *p = __float2half_rn(v);
    else
        *p = __float2bfloat16_rn(v);
}

// The residual operand at the position of a store: VG consecutive elements, or one, widened to fp32.
template <typename YT, int VG>
__device__ __forceinline__ void load_res_vec(const YT* p, float (&v)[VG])
{
    if constexpr (sizeof(YT) == 4) {
#pragma unroll
        for (int i = 0; i < VG / 4; ++i) {
            const float4 r = __ldg(reinterpret_cast<const float4*>(p) + i);
            v[4 * i] = r.x; v[4 * i + 1] = r.y; v[4 * i + 2] = r.z; v[4 * i + 3] = r.w;
        }
    } else if constexpr (std::is_same<YT, __half>::value) {
        __half2 h[VG / 2];
        if constexpr (VG == 8)
            *reinterpret_cast<uint4*>(h) = __ldg(reinterpret_cast<const uint4*>(p));
        else
            *reinterpret_cast<uint2*>(h) = __ldg(reinterpret_cast<const uint2*>(p));
#pragma unroll
        for (int i = 0; i < VG / 2; ++i) {
            const float2 f = __half22float2(h[i]);
            v[2 * i] = f.x; v[2 * i + 1] = f.y;
        }
    } else {
        __nv_bfloat162 h[VG / 2];
        if constexpr (VG == 8)
            *reinterpret_cast<uint4*>(h) = __ldg(reinterpret_cast<const uint4*>(p));
        else
            *reinterpret_cast<uint2*>(h) = __ldg(reinterpret_cast<const uint2*>(p));
#pragma unroll
        for (int i = 0; i < VG / 2; ++i) {
            const float2 f = __bfloat1622float2(h[i]);
            v[2 * i] = f.x; v[2 * i + 1] = f.y;
        }
    }
}

template <typename YT>
__device__ __forceinline__ float load_res_one(const YT* p)
{
    if constexpr (sizeof(YT) == 4)
        return __ldg(p);
    else if constexpr (std::is_same<YT, __half>::value)
        return __half2float(__ldg(p));
    else
        return __bfloat162float(__ldg(p));
}

// ---- producer: one warp copies (item, chunk) after (item, chunk) into the ring ---------------
// LDB = bytes per X copy.  Each lane owns NCOL fixed pixel vectors of the tile and walks the
// channels of the chunk, so its source pointers are computed once per item.
// XPAD = bytes of padding after each channel row of the tile in shared memory.
// GR = consumer groups: with 2, the items of the thread block belong alternately to group 0 and
// group 1, and each group has its own half of the ring (stages and barriers), so that a barrier
// is only ever used by one group, one phase after the other.
template <typename XT, int G, int P, int LDB, int XPAD = 0, int GR = 1>
__device__ __forceinline__ void produce(const ConvArgs& a, unsigned char* smem, int lane, int pw, int npw)
{
    constexpr int T = 32 * P;
    constexpr int SZ = (int)sizeof(XT);
    constexpr int ROWB = T * SZ + XPAD;
    constexpr int EV = LDB / SZ;            // elements per copy
    constexpr int VPR = T / EV;             // copies per channel row
    constexpr int NCOL = VPR >= 32 ? VPR / 32 : 1;   // copies per channel row per lane
    constexpr int RP = VPR >= 32 ? 1 : 32 / VPR;     // channel rows the warp covers per pass
    const int vlane = lane % VPR;           // (== lane when VPR >= 32)
    const int rlane = lane / VPR;           // first channel row of this lane (0 when VPR >= 32)

    const size_t ch_bytes = (size_t)a.hw * SZ;
    const uint32_t smem_u32 = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t ring = smem_u32 + 16 * kMaxStages;
    const int S = a.stages / GR;            // stages of one group's ring
    const int items = a.n_tiles * a.n_rg;
    int kk = 0;                             // running (item, chunk) counter = position in the group's ring
    int kk_other = 0, turn = 0;             // (GR == 2) the other group's counter; whose item this is

    bool dep_ok = false;                    // has the predecessor kernel been waited for yet?
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int tile = item / a.n_rg;
        const int rg = item - tile * a.n_rg;
        const int q0 = tile * T;
        const unsigned char* src[NCOL];
        bool ok[NCOL];
#pragma unroll
        for (int i = 0; i < NCOL; ++i) {
            const int q = q0 + (vlane + 32 * i) * EV;
            ok[i] = q < a.q_total;
            const int n = ok[i] ? q / a.hw : 0;
            const int p = ok[i] ? q - n * a.hw : 0;
            src[i] = static_cast<const unsigned char*>(a.x) + ((size_t)n * a.cin * a.hw + p) * SZ;
        }
        const int* slice = a.slice + rg * a.nch;
        const int* rowoff = a.rowoff + (size_t)rg * a.nch * a.ros;

        int sl_lo = 0, sl_hi = 0;           // slice bounds of chunks k0 + lane, fetched 32 chunks at a time
        for (int k = 0; k < a.nch; ++k, ++kk) {
            // (a load per chunk here would put a global-memory round trip in front of every stage's copies)
            if ((k & 31) == 0) {
                sl_lo = k + lane <= a.nch ? __ldg(slice + k + lane) : 0;
                sl_hi = k + lane + 1 <= a.nch ? __ldg(slice + k + lane + 1) : sl_lo;
            }
            const int s = turn * S + kk % S;
            if (kk >= S) {                  // wait until the consumers have released this stage
                if (!mbar_wait(smem_u32 + 8 * kMaxStages + 8 * s, ((kk / S) - 1) & 1)) {
                    if (lane == 0) atomicExch(a.err, kErrEmptyWait);
                    cp_async_wait_all();
                    return;
                }
            }
            const uint32_t st = ring + s * a.stage_bytes;
            // the row group's pair records of this chunk and their per-row offsets
            const int r0 = __shfl_sync(0xffffffffu, sl_lo, k & 31);
            const int n16 = __shfl_sync(0xffffffffu, sl_hi, k & 31) - r0;
            const unsigned char* rsrc = a.rec + (size_t)r0 * 16;
            for (int i = lane + 32 * pw; i < n16; i += 32 * npw) cp_async_16(st + a.off_rec + i * 16, rsrc + (size_t)i * 16);
            const int* osrc = rowoff + (size_t)k * a.ros;
            for (int i = lane + 32 * pw; i < a.ros / 4; i += 32 * npw) cp_async_16(st + a.off_rowoff + i * 16, osrc + 4 * i);
            // X (or its repacked copy) is the predecessor kernel's output: wait for it once, after the
            // first weight copies are already in flight
            if (!dep_ok) { grid_dep_wait(); dep_ok = true; }
            // X tile of this chunk
            const int cbase = k * a.kc;
            const int nrows = min(a.kc, a.cin - cbase);
#pragma unroll
            for (int i = 0; i < NCOL; ++i) {
                if (!ok[i]) continue;
                const unsigned char* sp = src[i] + (size_t)cbase * ch_bytes;
                const uint32_t dp = st + (vlane + 32 * i) * LDB;
                if constexpr (LDB == 16) {
                    for (int c = rlane + pw * RP; c < nrows; c += RP * npw) cp_async_16(dp + c * ROWB, sp + c * ch_bytes);
                } else if constexpr (LDB == 8) {
                    for (int c = rlane + pw * RP; c < nrows; c += RP * npw) cp_async_8(dp + c * ROWB, sp + c * ch_bytes);
                } else if constexpr (LDB == 4) {
                    for (int c = rlane + pw * RP; c < nrows; c += RP * npw) cp_async_4(dp + c * ROWB, sp + c * ch_bytes);
                } else {   // 2-byte elements at odd alignment: plain loads and shared-memory stores
                    unsigned char* d = smem + 16 * kMaxStages + s * a.stage_bytes + (vlane + 32 * i) * LDB;
                    for (int c = rlane + pw * RP; c < nrows; c += RP * npw)
                        *reinterpret_cast<unsigned short*>(d + c * ROWB) =
                            __ldg(reinterpret_cast<const unsigned short*>(sp + c * ch_bytes));
                }
            }
            if constexpr (LDB == 2) __threadfence_block();
            mbar_arrive_on_copies(smem_u32 + 8 * s);      // "full" completes when all producer lanes' copies land
        }
        if constexpr (GR == 2) {            // the next item is the other group's
            const int t = kk; kk = kk_other; kk_other = t;
            turn ^= 1;
        }
    }
    cp_async_wait_all();
}

// ---- producer, bulk-copy flavour ---------------------------------------------------------------
// Used when every (image, channel) row of X starts on a 16-byte boundary and is a multiple of 16
// bytes long.  One bulk copy moves a whole run of consecutive pixels of one channel (a tile row,
// split where the tile crosses from one image into the next); the lanes of the producer warp
// share the channel rows of the chunk.  Lane 0 announces the chunk's byte count on the "full"
// mbarrier, which completes when all of them have landed.
template <typename XT, int G, int P, int XPAD = 0, int GR = 1>
__device__ __forceinline__ void produce_bulk(const ConvArgs& a, unsigned char* smem, int lane, int pw, int npw)
{
    constexpr int T = 32 * P;
    constexpr int SZ = (int)sizeof(XT);
    constexpr int ROWB = T * SZ + XPAD;
    const size_t ch_bytes = (size_t)a.hw * SZ;
    const uint32_t smem_u32 = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t ring = smem_u32 + 16 * kMaxStages;
    const int S = a.stages / GR;            // stages of one group's ring
    const int items = a.n_tiles * a.n_rg;
    int kk = 0;
    int kk_other = 0, turn = 0;             // (GR == 2) the other group's counter; whose item this is

    bool dep_ok = false;                    // has the predecessor kernel been waited for yet?
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int tile = item / a.n_rg;
        const int rg = item - tile * a.n_rg;
        const int q0 = tile * T;
        const int vt = min(T, a.q_total - q0);          // valid pixels of this tile
        const int n0 = q0 / a.hw;
        const int p0 = q0 - n0 * a.hw;
        const unsigned char* xbase = static_cast<const unsigned char*>(a.x) + ((size_t)n0 * a.cin * a.hw + p0) * SZ;
        const int* slice = a.slice + rg * a.nch;
        const int* rowoff = a.rowoff + (size_t)rg * a.nch * a.ros;

        int sl_lo = 0, sl_hi = 0;           // slice bounds of chunks k0 + lane, fetched 32 chunks at a time
        for (int k = 0; k < a.nch; ++k, ++kk) {
            if ((k & 31) == 0) {
                sl_lo = k + lane <= a.nch ? __ldg(slice + k + lane) : 0;
                sl_hi = k + lane + 1 <= a.nch ? __ldg(slice + k + lane + 1) : sl_lo;
            }
            const int s = turn * S + kk % S;
            if (kk >= S) {
                if (!mbar_wait(smem_u32 + 8 * kMaxStages + 8 * s, ((kk / S) - 1) & 1)) {
                    if (lane == 0) atomicExch(a.err, kErrEmptyWait);
                    goto drain;
                }
            }
            {
                const uint32_t st = ring + s * a.stage_bytes;
                const uint32_t bar = smem_u32 + 8 * s;
                const int cbase = k * a.kc;
                const int nrows = min(a.kc, a.cin - cbase);
                const int r0 = __shfl_sync(0xffffffffu, sl_lo, k & 31);
                const int rbytes = (__shfl_sync(0xffffffffu, sl_hi, k & 31) - r0) * 16;
                const bool tiled = a.bulk == 2;
                if (lane == 0 && pw == 0)
                    mbar_arrive_expect_tx(bar, (uint32_t)(nrows * (tiled ? ROWB : vt * SZ) + rbytes + a.ros * 4));
                __syncwarp();
                if (lane == 0 && pw == 0 && rbytes > 0) bulk_copy_g2s(st + a.off_rec, a.rec + (size_t)r0 * 16, (uint32_t)rbytes, bar);
                if (lane == 1 && pw == 0)
                    bulk_copy_g2s(st + a.off_rowoff, rowoff + (size_t)k * a.ros, (uint32_t)(a.ros * 4), bar);
                // X (or its repacked copy) is the predecessor kernel's output: wait for it once,
                // after the first weight copies are already in flight
                if (!dep_ok) { grid_dep_wait(); dep_ok = true; }
                if (tiled) {
                    // the chunk's channel rows of this tile lie one after the other: copies of eight rows each
                    const unsigned char* src = static_cast<const unsigned char*>(a.x) + ((size_t)tile * a.cin + cbase) * ROWB;
                    const uint32_t total = (uint32_t)nrows * ROWB;
                    constexpr uint32_t PIECE = 8 * ROWB;
                    for (uint32_t o = (uint32_t)(lane + 32 * pw) * PIECE; o < total; o += 32u * npw * PIECE)
                        bulk_copy_g2s(st + o, src + o, min(PIECE, total - o), bar);
                }
                // X: channel rows lane, lane+32, ...; each row is one copy per image it touches
                for (int c = lane + 32 * pw; c < nrows && !tiled; c += 32 * npw) {
                    const unsigned char* src = xbase + (size_t)(cbase + c) * ch_bytes;
                    uint32_t dst = st + c * ROWB;
                    int left = vt, p = p0;
                    while (left > 0) {
                        const int len = min(a.hw - p, left);
                        bulk_copy_g2s(dst, src, (uint32_t)(len * SZ), bar);
                        dst += len * SZ;
                        // next image: same channel, pixel 0
                        src += (size_t)len * SZ + (size_t)(a.cin - 1) * ch_bytes;
                        left -= len;
                        p = 0;
                    }
                }

            }
        }
        if constexpr (GR == 2) {            // the next item is the other group's
            const int t = kk; kk = kk_other; kk_other = t;
            turn ^= 1;
        }
    }
drain:
    // Do not leave while copies of this warp may still be landing: wait (bounded) for the last
    // fills of every stage.
    for (int j = max(0, kk - S); j < kk; ++j) mbar_wait(smem_u32 + 8 * (turn * S + j % S), (j / S) & 1);
    if constexpr (GR == 2)
        for (int j = max(0, kk_other - S); j < kk_other; ++j) mbar_wait(smem_u32 + 8 * ((turn ^ 1) * S + j % S), (j / S) & 1);
}

// SPLIT: the flavour for schedules in which block rows are split into parts (the hand-over below); it is
// a compile-time flavour because even its few extra live values cost the common flavour spills.
template <typename XT, int G, int P, int RW, int NW, int MINB, int NPW, bool SPLIT = false>
__global__ void __launch_bounds__((NW + NPW) * 32, MINB) spconv1x1_kernel(const ConvArgs a)
{
    constexpr int T = 32 * P;                         // pixels per tile
    constexpr int SZ = (int)sizeof(XT);
    constexpr int VG = (P * SZ >= 16) ? 16 / SZ : P;  // elements per shared-memory vector load
    constexpr int NG = P / VG;                        // vector groups per lane
    // registers a thread may use, and whether the deep software pipeline fits in them
    // (the register file is handed out as if the block had a multiple of 128 threads)
    constexpr int kThreadsAlloc = ((NW + NPW) * 32 + 127) / 128 * 128;
    constexpr int kRegCap = 65536 / (kThreadsAlloc * MINB) > 255 ? 255 : 65536 / (kThreadsAlloc * MINB) / 8 * 8;
    constexpr bool kDeep = RW * G * P + 4 * G + 4 * P + 28 <= kRegCap;

    extern __shared__ __align__(16) unsigned char smem[];   // [full[8] | empty[8] | ring]

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int S = a.stages;
    const uint32_t smem_u32 = (uint32_t)__cvta_generic_to_shared(smem);

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32 + 8 * s, a.bulk ? 1 : 32 * NPW);     // full: one announcing arrival, or every producer lane
            mbar_init(smem_u32 + 8 * kMaxStages + 8 * s, NW);       // empty: one arrival per consumer warp
        }
        if constexpr (SPLIT) mbar_init(smem_u32 + a.off_xch, NW);  // hand-over of split rows: one arrival per consumer warp
    }
    __syncthreads();
    grid_dep_launch();

    if (warp >= NW) {   // ---- producer warps ------------------------------------------------
        const int pw = warp - NW;
        if (a.bulk) {
            produce_bulk<XT, G, P>(a, smem, lane, pw, NPW);
            return;
        }
        switch (a.ld_bytes) {
            case 16: produce<XT, G, P, 16>(a, smem, lane, pw, NPW); break;
            case 8: produce<XT, G, P, 8>(a, smem, lane, pw, NPW); break;
            case 4: produce<XT, G, P, 4>(a, smem, lane, pw, NPW); break;
            default:
                if constexpr (SZ == 2) produce<XT, G, P, 2>(a, smem, lane, pw, NPW);
                break;
        }
        return;
    }

    // ---- consumer warps ---------------------------------------------------------------------
    const unsigned char* ring = smem + 16 * kMaxStages;
    const int items = a.n_tiles * a.n_rg;
    int kk = 0;

    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int tile = item / a.n_rg;
        const int rg = item - tile * a.n_rg;
        const int q0 = tile * T;

        // local rows of this warp: tier s, dealt in serpentine order so that the warps' totals match
        int lrow[RW], rowid[RW];
#pragma unroll
        for (int s = 0; s < RW; ++s) {
            lrow[s] = s * NW + ((s & 1) ? NW - 1 - warp : warp);
            rowid[s] = lrow[s] < a.rpg ? __ldg(a.rowmap + rg * a.rpg + lrow[s]) : -1;
        }

        // bring the rows' bias values into L1 now, so that the epilogue does not start with a
        // global-memory round trip
        if (a.bias) {
#pragma unroll
            for (int s = 0; s < RW; ++s)
                if (rowid[s] >= 0 && lane == 0) {
                    const float* bp = a.bias + min(rowid[s] * G, a.cout - 1);
                    asm volatile("prefetch.global.L1 [%0];\n" ::"l"(bp));
                }
        }

        float2 acc[RW][G][P / 2];
#pragma unroll
        for (int s = 0; s < RW; ++s)
#pragma unroll
            for (int j = 0; j < G; ++j)
#pragma unroll
                for (int e = 0; e < P / 2; ++e) acc[s][j][e] = make_float2(0.0f, 0.0f);

        for (int k = 0; k < a.nch; ++k, ++kk) {
            const int st = kk % S;
            if (!mbar_wait(smem_u32 + 8 * st, (kk / S) & 1)) {      // chunk has landed in stage st
                if (lane == 0) atomicExch(a.err, kErrFullWait);
                return;
            }
            const unsigned char* stage = ring + st * a.stage_bytes;
            const unsigned char* xs = stage + lane * (VG * SZ);
            const unsigned char* recs = stage + a.off_rec;
            const int4* roff = reinterpret_cast<const int4*>(stage + a.off_rowoff);
#pragma unroll
            for (int s = 0; s < RW; ++s) {
                if (lrow[s] >= a.rpg) continue;
                const int4 hd = roff[lrow[s]];     // {segment start, first two columns, pairs}
                if (hd.w > 0) consume_segment<XT, G, P, kDeep>(acc[s], xs, recs + hd.x * 16, hd.w, hd.y, hd.z);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32 + 8 * kMaxStages + 8 * st);   // stage st may be refilled
        }

        // ---- rows split into parts: the secondary parts hand their partial sums to the primary one through
        // shared memory (two alternating sets of tiles, one bounded barrier among the consumer warps per item);
        // the primary adds them in slot order, so the result does not depend on timing
        if constexpr (SPLIT) {      // (every item takes the barrier, so its phase follows from the item's number)
            const int xphase = (item - (int)blockIdx.x) / (int)gridDim.x;
            const int xrg = item - (item / a.n_rg) * a.n_rg;
            constexpr int TILE2 = G * (P / 2) * 32;             // float2 elements of one hand-over tile
            float2* xch = reinterpret_cast<float2*>(smem + a.off_xch + 16) + (size_t)(xphase & 1) * a.xch_slots * TILE2;
#pragma unroll
            for (int s = 0; s < RW; ++s) {
                const int lr = s * NW + ((s & 1) ? NW - 1 - warp : warp);
                const int uw = lr < a.rpg ? __ldg(a.unit + xrg * a.rpg + lr) : 0;
                if ((uw & 15) == 2) {
                    float2* t = xch + (size_t)((uw >> 4) & 0xfff) * TILE2 + lane;
#pragma unroll
                    for (int j = 0; j < G; ++j)
#pragma unroll
                        for (int e = 0; e < P / 2; ++e) t[(j * (P / 2) + e) * 32] = acc[s][j][e];
                    rowid[s] = -1;                              // a secondary part stores nothing itself
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32 + a.off_xch);
            if (!mbar_wait(smem_u32 + a.off_xch, xphase & 1)) {
                if (lane == 0) atomicExch(a.err, kErrFullWait);
                return;
            }
#pragma unroll
            for (int s = 0; s < RW; ++s) {
                const int lr = s * NW + ((s & 1) ? NW - 1 - warp : warp);
                const int uw = lr < a.rpg ? __ldg(a.unit + xrg * a.rpg + lr) : 0;
                if ((uw & 15) == 1) {
                    const int first = (uw >> 4) & 0xfff, count = uw >> 16;
                    for (int i = 0; i < count; ++i) {
                        const float2* t = xch + (size_t)(first + i) * TILE2 + lane;
#pragma unroll
                        for (int j = 0; j < G; ++j)
#pragma unroll
                            for (int e = 0; e < P / 2; ++e) {
                                const float2 v = t[(j * (P / 2) + e) * 32];
                                acc[s][j][e].x += v.x;
                                acc[s][j][e].y += v.y;
                            }
                    }
                }
            }
        }

        // ---- epilogue: bias, ReLU, store ----------------------------------------------------
        grid_dep_wait();    // (long satisfied: the data consumed above was loaded after the producer's wait)
        // (the residual operand is a compile-time flavour of the epilogue, so that layers without one
        // run exactly the code they would run if the operand did not exist)
        auto epilogue = [&](auto* ybase, auto has_res) {
            using YT = std::remove_pointer_t<decltype(ybase)>;
            constexpr bool RES = decltype(has_res)::value;
            size_t yoff[NG];
            bool yok[NG];
            int yn[NG], yp[NG];
#pragma unroll
            for (int gi = 0; gi < NG; ++gi) {
                const int q = q0 + gi * (32 * VG) + lane * VG;
                yok[gi] = q < a.q_total;
                yn[gi] = q / a.hw;
                yp[gi] = q - yn[gi] * a.hw;
                yoff[gi] = (size_t)yn[gi] * a.cout * a.hwy + yp[gi];
            }
#pragma unroll
            for (int s = 0; s < RW; ++s) {
                if (rowid[s] < 0) continue;
#pragma unroll
                for (int j = 0; j < G; ++j) {
                    const int co = rowid[s] * G + j;
                    if (co >= a.cout) continue;
                    const float bv = a.bias ? __ldg(a.bias + co) : 0.0f;
#pragma unroll
                    for (int gi = 0; gi < NG; ++gi) {
                        float v[VG];
#pragma unroll
                        for (int t = 0; t < VG; ++t) {
                            const float2 a2 = acc[s][j][(gi * VG + t) / 2];
                            v[t] = (((gi * VG + t) & 1) ? a2.y : a2.x) + bv;
                            if constexpr (!RES) {
                                if (a.relu) v[t] = fmaxf(v[t], 0.0f);
                            }
                        }
                        const YT* rbase = static_cast<const YT*>(a.res);
                        if (a.st_vec) {
                            if (yok[gi]) {
                                const size_t o = yoff[gi] + (size_t)co * a.hwy;
                                if constexpr (RES) {
                                    float r[VG];
                                    load_res_vec<YT, VG>(rbase + o, r);
#pragma unroll
                                    for (int t = 0; t < VG; ++t) {
                                        v[t] += r[t];
                                        if (a.relu) v[t] = fmaxf(v[t], 0.0f);
                                    }
                                }
                                store_vec<YT, VG>(ybase + o, v);
                            }
                        } else if (a.st_grp) {
                            // the lane's VG pixels lie in one image (the row length of X, padded or not,
                            // is a multiple of VG); pixels p >= hwy exist only as padding of the repacked X
                            if (yok[gi]) {
                                const size_t o = yoff[gi] + (size_t)co * a.hwy;
#pragma unroll
                                for (int t = 0; t < VG; ++t)
                                    if (yp[gi] + t < a.hwy) {
                                        float u = v[t];
                                        if constexpr (RES) {
                                            u += load_res_one<YT>(rbase + o + t);
                                            if (a.relu) u = fmaxf(u, 0.0f);
                                        }
                                        store_one<YT>(ybase + o + t, u);
                                    }
                            }
                        } else {
                            // element by element: the run may cross into the next image, and pixels
                            // p >= hwy exist only as padding of the repacked X
                            int nn = yn[gi], pp = yp[gi];
#pragma unroll
                            for (int t = 0; t < VG; ++t) {
                                while (pp >= a.hw) { pp -= a.hw; ++nn; }
                                if (q0 + gi * (32 * VG) + lane * VG + t < a.q_total && pp < a.hwy) {
                                    const size_t o = ((size_t)nn * a.cout + co) * a.hwy + pp;
                                    float u = v[t];
                                    if constexpr (RES) {
                                        u += load_res_one<YT>(rbase + o);
                                        if (a.relu) u = fmaxf(u, 0.0f);
                                    }
                                    store_one<YT>(ybase + o, u);
                                }
                                ++pp;
                            }
                        }
                    }
                }
            }
        };
        auto run_epilogue = [&](auto* ybase) {
            if (a.res) epilogue(ybase, std::true_type{});
            else epilogue(ybase, std::false_type{});
        };
        if constexpr (sizeof(XT) == 4) {
            run_epilogue(static_cast<float*>(a.y));
        } else {
            if (a.y_f32) run_epilogue(static_cast<float*>(a.y));
            else run_epilogue(static_cast<XT*>(a.y));
        }
    }
}

// One entry of the table of compiled kernel variants.
// mma = 1: the tensor-core kernel (fp16 only), which takes the step-record flavour of the schedule.
struct KernelVariant {
    int is_f16;     // the alcs_dtype the kernel takes: 0 fp32, 1 binary16, 2 bfloat16
    int g, p, rw, nw, minb, npw;
    const void* fn;
    int mma;
    int groups;     // consumer groups that take the items of a thread block in turn (1 or 2); nw counts all consumer warps
    int split;      // 1: takes schedules in which long block rows are split into parts
};

#define ALCS_VARIANT_P(XT, ISF16, G, P, RW, NW, MINB, NPW) \
    {ISF16, G, P, RW, NW, MINB, NPW, (const void*)&spconv1x1_kernel<XT, G, P, RW, NW, MINB, NPW>, 0, 1}
#define ALCS_VARIANT(XT, ISF16, G, P, RW, NW, MINB) ALCS_VARIANT_P(XT, ISF16, G, P, RW, NW, MINB, 1)
#define ALCS_VARIANT_SPLIT(XT, ISF16, G, P, RW, NW, MINB, NPW) \
    {ISF16, G, P, RW, NW, MINB, NPW, (const void*)&spconv1x1_kernel<XT, G, P, RW, NW, MINB, NPW, true>, 0, 1, 1}

// Defined one per translation unit, concatenated by alcs_device.cu.
const KernelVariant* variants_f32_g4(int* n);
const KernelVariant* variants_f32_other(int* n);
const KernelVariant* variants_f16(int* n);
const KernelVariant* variants_f16_mma(int* n);
const KernelVariant* variants_bf16(int* n);

}  // namespace alcs

#endif  // ALCS_KERNELS_CUH_
