// Device code of the general k_h x k_w SIMD-structured sparse convolution for sm_100a.
//
// The paper's Section 3.2.2 views the convolution as W* x I*: W* stacks the flattened filters
// (column = (c, r, s)), I* stacks the vectorised input patches, and the grouped-CSR format stores,
// per group of g filters, the kept columns of W*.  The multiply loop is the same as for 1x1
// kernels (zero the accumulators, walk the group's kept columns, multiply the column's g weights
// with the input vector the column offset addresses); what changes is what a column addresses:
// the input image of channel c shifted by the tap (r, s).  I* is never materialised.
//
//   work item    = (image, strip of TH output rows, row group); for images of at most 64 output
//                  positions, (2 or 4 whole images, row group)
//   thread block = persistent; per item it stages the input patch that the strip needs (halo and
//                  zero padding included) in shared memory -- all input channels at once where
//                  they fit, else chunk of channels after chunk -- and its warps multiply
//   patch layout = per channel, stride x stride "parity planes": input pixel (ih, iw) of the
//                  patch window lies in plane (ih % stride, iw % stride) at [ih / stride][iw / stride],
//                  planes have PR rows of pitch WP words.  With that layout the address of the
//                  input that output position (oh, ow) needs for column (c, r, s) is
//                      coloff(c, r, s) + (oh * WP + ow),      coloff = c*CHW + plane(r,s)*PL + (r/stride)*WP + s/stride
//                  for every stride: a per-column constant plus a per-position constant.  The
//                  per-column constants are baked into the launch schedule as byte offsets.
//   position     = j = oh_local * WP + ow, 0 <= j < TH*WP.  Positions with ow >= OW (the
//                  (kw-1)/stride extra columns of the pitch) are computed and not stored.
//   warp         = one tile of 32*P consecutive positions (lane owns j0 + lane + 32*t, so every
//                  shared-memory load is 32 consecutive words) x one block row at a time; the
//                  warps that share a position tile take the row group's rows from a shared
//                  counter, longest rows first.  G*P fp32 accumulators per lane.
//   weights      = pair records (two byte offsets of the NEXT pair, the 2*G values of this pair);
//                  each row is one contiguous run in global memory, which its warp streams
//                  through a private shared-memory double buffer with cp.async.
//
// There are no cross-warp waits other than __syncthreads, so nothing here can spin.
#ifndef ALCS_CONV2D_CUH_
#define ALCS_CONV2D_CUH_

#include <utility>

#include "alcs_kernels.cuh"

namespace alcs {

struct Conv2dArgs {
    const float* x;            // [n][cin][h][wd]
    float* y;                  // [n][cout][oh][ow]
    const float* bias;         // [cout] or nullptr
    const unsigned char* rec;  // pair records, [row group][local row]
    const int* slice;          // [n_rg + 1] start of each row group's records, 16-byte units
    const int* rowoff;         // [n_rg][rpg] int4 {row start inside the slice (16-byte units), first two byte offsets, pairs}
    const int* rowmap;         // [n_rg][rpg] block row of each local row, -1 = none
    int rows, cin, cout;
    int h, wd, oh, ow;
    int kh, kw, pad;
    int th;                    // output rows per strip
    int n_strips, n_rg, rpg, n_img;
    int wp, pr, pl, chw;       // plane pitch, plane rows, words per plane, words per channel and image
    int chs;                   // words per channel of the staged patch = images per item * chw
    int n_igrp;                // groups of NI images = work items per (strip, row group)
    int npt, nrs;              // position tiles per strip, warps per position tile
    int kc, nch;               // input channels per chunk, number of chunks
    int slack;                 // words after the patch that out-of-strip positions may read
    int off_wbuf;              // byte offset of the warps' record buffers in shared memory (16-byte aligned)
    int relu;
};

// Shared-memory loads by 32-bit shared-space address (no generic-pointer arithmetic in the hot loop).
// The P positions a lane owns of the input row a column addresses: xs = shared address of the
// lane's first position, byte_off = the column's offset; positions are 32 words apart.
template <int OFF>
__device__ __forceinline__ float lds_off(uint32_t p)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1 + %2];\n" : "=f"(v) : "r"(p), "n"(OFF));
    return v;
}
// Position t of a lane (t < P) belongs to image t / M of the work item's NI images, M = P / NI, and is
// position lane + 32 * (t % M) inside it: which image and which immediate offset are compile-time
// facts, so a column costs NI address additions and P loads.
template <int P, int NI, int... T>
__device__ __forceinline__ void load_x2d_seq(const uint32_t (&p)[NI], float2 (&x)[P / 2], std::integer_sequence<int, T...>)
{
    constexpr int M = P / NI;
    ((x[T].x = lds_off<128 * ((2 * T) % M)>(p[(2 * T) / M]), x[T].y = lds_off<128 * ((2 * T + 1) % M)>(p[(2 * T + 1) / M])), ...);
}
template <int P, int NI>
__device__ __forceinline__ void load_x2d(const uint32_t (&xs)[NI], int byte_off, float2 (&x)[P / 2])
{
    uint32_t p[NI];
#pragma unroll
    for (int i = 0; i < NI; ++i) p[i] = xs[i] + (uint32_t)byte_off;
    load_x2d_seq<P, NI>(p, x, std::make_integer_sequence<int, P / 2>{});
}

__device__ __forceinline__ float4 lds_v4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// One pair record from shared memory by shared-space address (same layout as load_record).
template <int G>
__device__ __forceinline__ void load_record_s(uint32_t p, int& c0, int& c1, float (&w0)[G], float (&w1)[G])
{
    const float4 h = lds_v4(p);
    c0 = __float_as_int(h.x);
    c1 = __float_as_int(h.y);
    if constexpr (G == 1) {
        w0[0] = h.z;
        w1[0] = h.w;
    } else if constexpr (G == 2) {
        const float4 v = lds_v4(p + 16);
        w0[0] = v.x; w0[1] = v.y; w1[0] = v.z; w1[1] = v.w;
    } else {
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 v = lds_v4(p + 16 + 16 * i);
            w0[4 * i] = v.x; w0[4 * i + 1] = v.y; w0[4 * i + 2] = v.z; w0[4 * i + 3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 v = lds_v4(p + 16 + 4 * G + 16 * i);
            w1[4 * i] = v.x; w1[4 * i + 1] = v.y; w1[4 * i + 2] = v.z; w1[4 * i + 3] = v.w;
        }
    }
}

// 4-byte asynchronous copy global -> shared; src_bytes = 0 writes zero without reading src.
__device__ __forceinline__ void cp_async_4_zfill(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// Records of one warp travel through a private shared-memory double buffer: rec_batch(g) records
// (600 to 800 bytes) per half, copied with 16-byte cp.async, so the hot loop reads them as
// shared-memory broadcasts (as the pointwise kernel does) instead of waiting for L2.
__host__ __device__ constexpr int rec_batch(int g) { return g <= 4 ? 16 : g == 8 ? 8 : 4; }
__host__ __device__ constexpr int rec_buffer_bytes(int g) { return 2 * rec_batch(g) * record_bytes(g); }

// Multiply-accumulate `n` pair records that lie in shared memory at rp; (oa0, oa1) = byte offsets of
// the first pair's columns on entry and of the pair after the last one on return.  Same
// two-register-set rotation as the pointwise kernel: the record and the input vectors of pair i+1
// are loaded while pair i is multiplied.
template <int G, int P, int NI>
__device__ __forceinline__ void consume_batch2d(float2 (&acc)[G][P / 2], const uint32_t (&xs)[NI], uint32_t rp, int n,
                                                int& oa0, int& oa1)
{
    constexpr int REC = record_bytes(G);
    if constexpr (G <= 4) {
        int ob0 = 0, ob1 = 0;
        float wA0[G], wA1[G], wB0[G], wB1[G];
        float2 xA0[P / 2], xA1[P / 2], xB0[P / 2], xB1[P / 2];
        load_record_s<G>(rp, ob0, ob1, wA0, wA1);
        load_x2d<P, NI>(xs, oa0, xA0);
        load_x2d<P, NI>(xs, oa1, xA1);
        int left = n;                       // pairs not yet multiplied, A is loaded
        while (true) {
            const bool moreB = left > 1;
            if (moreB) {
                load_record_s<G>(rp + REC, oa0, oa1, wB0, wB1);
                load_x2d<P, NI>(xs, ob0, xB0);
                load_x2d<P, NI>(xs, ob1, xB1);
            }
            fma_block<G, P>(acc, wA0, xA0);
            fma_block<G, P>(acc, wA1, xA1);
            if (!moreB) { oa0 = ob0; oa1 = ob1; break; }      // A was the last: its header names the next pair
            const bool moreA = left > 2;
            if (moreA) {
                load_record_s<G>(rp + 2 * REC, ob0, ob1, wA0, wA1);
                load_x2d<P, NI>(xs, oa0, xA0);
                load_x2d<P, NI>(xs, oa1, xA1);
            }
            fma_block<G, P>(acc, wB0, xB0);
            fma_block<G, P>(acc, wB1, xB1);
            if (!moreA) break;                                // B was the last: (oa0, oa1) came from its header
            rp += 2 * REC;
            left -= 2;
        }
    } else {
        // wide groups: the accumulators fill most of the register file; only the next pair's
        // offsets are fetched ahead
        for (int i = 0; i < n; ++i, rp += REC) {
            float2 x0[P / 2], x1[P / 2];
            float w[G];
            load_x2d<P, NI>(xs, oa0, x0);
            load_x2d<P, NI>(xs, oa1, x1);
            const float4 nx = lds_v4(rp);
#pragma unroll
            for (int q = 0; q < G / 4; ++q) {
                const float4 v = lds_v4(rp + 16 + 16 * q);
                w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
            }
            fma_block<G, P>(acc, w, x0);
#pragma unroll
            for (int q = 0; q < G / 4; ++q) {
                const float4 v = lds_v4(rp + 16 + 4 * G + 16 * q);
                w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
            }
            fma_block<G, P>(acc, w, x1);
            oa0 = __float_as_int(nx.x);
            oa1 = __float_as_int(nx.y);
        }
    }
}

// A FULL batch of rec_batch(G) (an even number of) pair records: the same rotation without any loop
// test, fully unrolled, so that the only branches left in the steady state are the batch loop's.
template <int G, int P, int NI>
__device__ __forceinline__ void consume_full_batch2d(float2 (&acc)[G][P / 2], const uint32_t (&xs)[NI], uint32_t rp,
                                                     int& oa0, int& oa1)
{
    constexpr int REC = record_bytes(G);
    constexpr int N = rec_batch(G);
    static_assert(N % 2 == 0, "the unrolled rotation handles the records two by two");
    if constexpr (G <= 4) {
        int ob0 = 0, ob1 = 0;
        float wA0[G], wA1[G], wB0[G], wB1[G];
        float2 xA0[P / 2], xA1[P / 2], xB0[P / 2], xB1[P / 2];
        load_record_s<G>(rp, ob0, ob1, wA0, wA1);
        load_x2d<P, NI>(xs, oa0, xA0);
        load_x2d<P, NI>(xs, oa1, xA1);
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            load_record_s<G>(rp + (2 * i + 1) * REC, oa0, oa1, wB0, wB1);
            load_x2d<P, NI>(xs, ob0, xB0);
            load_x2d<P, NI>(xs, ob1, xB1);
            fma_block<G, P>(acc, wA0, xA0);
            fma_block<G, P>(acc, wA1, xA1);
            if (i + 1 < N / 2) {
                load_record_s<G>(rp + (2 * i + 2) * REC, ob0, ob1, wA0, wA1);
                load_x2d<P, NI>(xs, oa0, xA0);
                load_x2d<P, NI>(xs, oa1, xA1);
            }
            fma_block<G, P>(acc, wB0, xB0);
            fma_block<G, P>(acc, wB1, xB1);
        }
        // (oa0, oa1) now hold the header of the last record: the columns of the pair after the batch
    } else {
        consume_batch2d<G, P, NI>(acc, xs, rp, N, oa0, oa1);
    }
}

// Multiply-accumulate one whole block row (or its segment inside a channel chunk): `npairs` pair
// records starting at rp in GLOBAL memory, streamed through this warp's double buffer `wbuf`.
template <int G, int P, int NI>
__device__ __forceinline__ void consume_row2d(float2 (&acc)[G][P / 2], const uint32_t (&xs)[NI], const unsigned char* rp,
                                              int npairs, int oa0, int oa1, uint32_t wbuf_u32, int lane)
{
    constexpr int REC = record_bytes(G);
    constexpr int kRecBatch = rec_batch(G);
    constexpr int HALF = kRecBatch * REC;
    const int nb = (npairs + kRecBatch - 1) / kRecBatch;
    auto fetch = [&](int b) {
        const int bytes = min(kRecBatch, npairs - b * kRecBatch) * REC;
        const unsigned char* src = rp + (size_t)b * HALF;
        const uint32_t dst = wbuf_u32 + (b & 1) * HALF;
        for (int o = lane * 16; o < bytes; o += 512) cp_async_16(dst + o, src + o);
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    };
    fetch(0);
    for (int b = 0; b < nb; ++b) {
        if (b + 1 < nb) {
            fetch(b + 1);
            asm volatile("cp.async.wait_group 1;\n" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        }
        __syncwarp();
        const int nrec = min(kRecBatch, npairs - b * kRecBatch);
        if (nrec == kRecBatch) consume_full_batch2d<G, P, NI>(acc, xs, wbuf_u32 + (b & 1) * HALF, oa0, oa1);
        else consume_batch2d<G, P, NI>(acc, xs, wbuf_u32 + (b & 1) * HALF, nrec, oa0, oa1);
        __syncwarp();           // every lane has read this half before the fetch after next refills it
    }
}

// G = group size, P = positions per lane, ST = stride (1 or 2), NW = warps per thread block,
// CHUNKED = which of the two ways through a work item this instance takes, NI = images per work item
// (small images: NI > 1 puts NI whole images, each padded to 32 * P / NI positions, into one position
// tile, so that a lane still owns P positions).
//
// Two ways through a work item.  With all input channels in one chunk (nch == 1) the warps that
// share a position tile take block rows from a shared counter, one row at a time.  With the
// channels split into nch chunks (patches too large for shared memory otherwise) every warp owns
// ONE block row of the row group for the whole item, keeps its accumulators across the chunks, and
// the block walks stage -> multiply -> stage -> ... ; the schedule then holds one segment per
// (row group, chunk, row) with chunk-local offsets.
template <int G, int P, int ST, int NW, bool CHUNKED, int NI>
__global__ void __launch_bounds__(NW * 32, 1) spconv2d_kernel(const Conv2dArgs a)
{
    extern __shared__ __align__(16) float patch[];     // [kc][ST*ST][pr][wp], a.slack words, then the warps' record buffers
    __shared__ int next_row[NW];                        // per position tile: next local row to take

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    constexpr int M = P / NI;                           // positions per lane and image
    const int items = a.n_igrp * a.n_strips * a.n_rg;
    const int patch_words = a.kc * a.chs;
    const uint32_t patch_u32 = (uint32_t)__cvta_generic_to_shared(patch);
    const int positions = a.th * a.wp;

    // the slack that positions past the last strip row, and the extra columns of the pitch, read
    for (int i = tid; i < a.slack; i += NW * 32) patch[patch_words + i] = 0.0f;

    const int pt = warp % a.npt;                        // position tile of this warp
    const int rs = warp / a.npt;                        // its slot among the warps of that tile
    const bool active = warp < a.npt * a.nrs;
    const int jbase = pt * (32 * P) + lane;
    const uint32_t wbuf = patch_u32 + a.off_wbuf + warp * rec_buffer_bytes(G);
    // shared address of the lane's first position of each image (positions past the end of a strip
    // or image read on into the next image, channel or the slack: in bounds, never stored)
    uint32_t xs[NI];
#pragma unroll
    for (int i = 0; i < NI; ++i) xs[i] = patch_u32 + 4u * (uint32_t)(NI == 1 ? jbase : i * a.chw + lane);

    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int rg = item % a.n_rg;
        const int strip = (item / a.n_rg) % a.n_strips;
        const int img = item / (a.n_rg * a.n_strips) * NI;      // first image of the item
        const int oh0 = strip * a.th;
        const float* ximg = a.x + (size_t)img * a.cin * a.h * a.wd;
        float* yimg = a.y + (size_t)img * a.cout * a.oh * a.ow;

        // where this lane's positions go in Y (-1: not an output)
        int yoff[P];
#pragma unroll
        for (int t = 0; t < P; ++t) {
            const int j = NI == 1 ? jbase + 32 * t : lane + 32 * (t % M);
            const int ol = j / a.wp;
            const int ow = j - ol * a.wp;
            const bool ok = j < positions && ow < a.ow && oh0 + ol < a.oh && img + t / M < a.n_img;
            yoff[t] = ok ? (NI == 1 ? 0 : (t / M) * a.cout * a.oh * a.ow) + (oh0 + ol) * a.ow + ow : -1;
        }

        // stage channels [c0, c0 + nc) of the strip's input window: one (channel, input row) per warp
        // and pass, lanes along the row, asynchronous 4-byte copies (zero-filled outside the image)
        // so that all of a warp's loads are in flight at once
        auto stage = [&](int c0, int nc) {
            const int ph_in = ST * a.pr, pw_in = ST * a.wp;
            const int ih0 = oh0 * ST - a.pad;
            if (pw_in > 16) {
                // wide rows: one (channel, image, input row) per warp and pass, lanes along the row.  What
                // depends only on the column (source column, destination offset, inside the image or not)
                // is worked out once per call; the row index advances without divisions.
                constexpr int kPass = 4;                            // columns per lane handled from registers
                int col_src[kPass];
                uint32_t col_dst[kPass];
                bool col_in[kPass], col_ok[kPass];
#pragma unroll
                for (int k = 0; k < kPass; ++k) {
                    const int cc = lane + 32 * k;
                    col_in[k] = cc < pw_in;
                    col_src[k] = cc - a.pad;
                    col_ok[k] = col_in[k] && col_src[k] >= 0 && col_src[k] < a.wd;
                    col_dst[k] = 4u * (uint32_t)((cc % ST) * a.pl + cc / ST);
                }
                const int total = nc * NI * ph_in;
                int c = warp / (NI * ph_in);
                int il = (warp - c * (NI * ph_in)) / ph_in;
                int rr = warp - (c * NI + il) * ph_in;
                for (int idx = warp; idx < total; idx += NW) {
                    if (NI == 1 || img + il < a.n_img) {            // (a missing image's slots keep stale values: never stored)
                        const int ih = ih0 + rr;
                        const bool row_ok = ih >= 0 && ih < a.h;
                        const float* src = ximg + (((size_t)il * a.cin + c0 + c) * a.h + (row_ok ? ih : 0)) * a.wd;
                        const uint32_t dst = patch_u32 + 4u * (uint32_t)(c * a.chs + il * a.chw + ((rr % ST) * ST) * a.pl + (rr / ST) * a.wp);
#pragma unroll
                        for (int k = 0; k < kPass; ++k) {
                            if (!col_in[k]) continue;
                            const bool ok = row_ok && col_ok[k];
                            cp_async_4_zfill(dst + col_dst[k], ok ? src + col_src[k] : ximg, ok ? 4 : 0);
                        }
                        for (int cc = lane + 32 * kPass; cc < pw_in; cc += 32) {      // images wider than 128 columns
                            const int iw = cc - a.pad;
                            const bool ok = row_ok && iw >= 0 && iw < a.wd;
                            cp_async_4_zfill(dst + 4u * (uint32_t)((cc % ST) * a.pl + cc / ST), ok ? src + iw : ximg, ok ? 4 : 0);
                        }
                    }
                    rr += NW;
                    while (rr >= ph_in) {
                        rr -= ph_in;
                        if (++il == NI) { il = 0; ++c; }
                    }
                }
            } else {
                // narrow rows (small images): one (channel, image) window per warp and pass, lanes over
                // all of its rows and columns, so that most lanes have an element to copy
                const int win = ph_in * pw_in;
                for (int idx = warp; idx < nc * NI; idx += NW) {
                    const int c = idx / NI;
                    const int il = idx - c * NI;
                    if (NI > 1 && img + il >= a.n_img) continue;
                    const float* src = ximg + ((size_t)il * a.cin + c0 + c) * a.h * a.wd;
                    const uint32_t dst = patch_u32 + 4u * (uint32_t)(c * a.chs + il * a.chw);
                    for (int e = lane; e < win; e += 32) {
                        const int rr = e / pw_in;
                        const int cc = e - rr * pw_in;
                        const int ih = ih0 + rr, iw = cc - a.pad;
                        const bool ok = ih >= 0 && ih < a.h && iw >= 0 && iw < a.wd;
                        cp_async_4_zfill(dst + 4u * (uint32_t)(((rr % ST) * ST + cc % ST) * a.pl + (rr / ST) * a.wp + cc / ST),
                                         ok ? src + ih * a.wd + iw : ximg, ok ? 4 : 0);
                    }
                }
            }
            cp_async_wait_all();
        };

        auto epilogue = [&](int row, float2 (&acc)[G][P / 2]) {
#pragma unroll
            for (int j = 0; j < G; ++j) {
                const int co = row * G + j;
                if (co >= a.cout) continue;
                const float bv = a.bias ? __ldg(a.bias + co) : 0.0f;
                float* yc = yimg + (size_t)co * a.oh * a.ow;
#pragma unroll
                for (int t = 0; t < P; ++t) {
                    const float2 a2 = acc[j][t / 2];
                    float v = ((t & 1) ? a2.y : a2.x) + bv;
                    if (a.relu) v = fmaxf(v, 0.0f);
                    if (yoff[t] >= 0) yc[yoff[t]] = v;
                }
            }
        };

        if constexpr (!CHUNKED) {
            __syncthreads();                            // everyone is done with the previous patch
            if (tid < NW) next_row[tid] = 0;
            stage(0, a.cin);
            __syncthreads();
            if (!active) continue;
            const int4* rowoff = reinterpret_cast<const int4*>(a.rowoff) + (size_t)rg * a.rpg;
            const unsigned char* recs = a.rec + (size_t)__ldg(a.slice + rg) * 16;
            while (true) {
                int lr = 0;
                if (lane == 0) lr = atomicAdd(&next_row[pt], 1);
                lr = __shfl_sync(0xffffffffu, lr, 0);
                if (lr >= a.rpg) break;
                const int row = __ldg(a.rowmap + rg * a.rpg + lr);
                if (row < 0) continue;
                const int4 hd = __ldg(rowoff + lr);
                float2 acc[G][P / 2];
#pragma unroll
                for (int j = 0; j < G; ++j)
#pragma unroll
                    for (int e = 0; e < P / 2; ++e) acc[j][e] = make_float2(0.0f, 0.0f);
                if (hd.w > 0) {
                    const unsigned char* rp = recs + (size_t)hd.x * 16;
                    consume_row2d<G, P, NI>(acc, xs, rp, hd.w, hd.y, hd.z, wbuf, lane);
                }
                epilogue(row, acc);
            }
        } else {
            // one block row per warp, accumulators kept across the channel chunks
            const int row = (active && rs < a.rpg) ? __ldg(a.rowmap + rg * a.rpg + rs) : -1;
            float2 acc[G][P / 2];
#pragma unroll
            for (int j = 0; j < G; ++j)
#pragma unroll
                for (int e = 0; e < P / 2; ++e) acc[j][e] = make_float2(0.0f, 0.0f);
            for (int k = 0; k < a.nch; ++k) {
                __syncthreads();                        // everyone is done with the previous chunk
                stage(k * a.kc, min(a.kc, a.cin - k * a.kc));
                __syncthreads();
                if (row < 0) continue;
                const int4 hd = __ldg(reinterpret_cast<const int4*>(a.rowoff) + ((size_t)rg * a.nch + k) * a.rpg + rs);
                if (hd.w > 0) {
                    const unsigned char* rp = a.rec + ((size_t)__ldg(a.slice + rg * a.nch + k) + hd.x) * 16;
                    consume_row2d<G, P, NI>(acc, xs, rp, hd.w, hd.y, hd.z, wbuf, lane);
                }
            }
            if (row >= 0) epilogue(row, acc);
        }
    }
}

// Launch the compiled variant for (g, positions per lane, stride); defined in alcs_conv2d.cu.
// Returns false if there is no such variant.  The first use of a variant raises its dynamic
// shared-memory limit.
constexpr int kConv2dWarps = 16;
// dynamic shared memory a block may ask for: the 227 KB per-block limit minus the kernel's static part
constexpr int kConv2dMaxDynSmem = 227 * 1024 - 256;
bool conv2d_variant_exists(int g, int p, int stride, int ni);
cudaError_t launch_conv2d(int g, int p, int stride, int ni, const Conv2dArgs& a, unsigned grid, size_t smem, cudaStream_t st);

}  // namespace alcs

#endif  // ALCS_CONV2D_CUH_
