// Device code of the SIMD-structured sparse pointwise convolution for sm_100a.
//
// Work decomposition (see the paper's Section 3.2.2, "Efficient multiplication computation", for
// the loop this re-creates: zero the accumulators, loop over a group's kept columns, multiply the
// column's g weights with the input vector addressed by the column offset, accumulate):
//
//   thread block = one tile of T = 32*P consecutive pixels (pixels of all images flattened,
//                  q = n*HW + p) x one slice of block rows ("row group")
//   warp         = RW block rows at a time, all T pixels of the tile
//   lane         = P pixels of each of those rows: G*P fp32 accumulators per row in registers
//
// The input channels are walked in chunks of KC channels.  Each chunk of the X tile
// ([KC][T] elements) is staged in shared memory by cp.async through a multi-stage ring, so the
// copy of chunk k+stages-1 overlaps the arithmetic of chunk k.  Inside a chunk a warp walks the
// (row, chunk) segment of the column list: column indices and weights are warp-uniform global
// loads (one broadcast transaction each), X values are 128-bit conflict-free shared-memory
// loads, and every X word feeds G FMAs.
#ifndef ALCS_KERNELS_CUH_
#define ALCS_KERNELS_CUH_

#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <type_traits>

namespace alcs {

struct ConvArgs {
    const void* x;            // [n][cin][hw] of XT
    void* y;                  // [n][cout][hw] of XT, or float if y_f32
    const float* bias;        // [cout] or nullptr
    const int* seg_ptr;       // [rows][nch+1]
    const int* cols;          // [nbp] chunk-local column
    const float* vals;        // [nbp][G]
    const int* row_order;     // [rows]
    int rows, cin, cout, hw;
    int q_total;              // n * hw
    int n_rg, rows_per_rg;    // row groups per pixel tile, block rows per row group
    int kc, nch, stages;
    int relu;
    int y_f32;                // only meaningful for XT = __half
    int ld_bytes;             // bytes per staging copy: 16, 8, 4 or 2
    int st_vec;               // 1 if vector stores are allowed
};

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
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;\n" ::: "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
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

// Weights of two consecutive blocks (2*G floats, 8- or 16-byte aligned), warp-uniform address.
template <int G>
__device__ __forceinline__ void load_w2(const float* __restrict__ p, float (&w0)[G], float (&w1)[G])
{
    if constexpr (G == 1) {
        const float2 v = __ldg(reinterpret_cast<const float2*>(p));
        w0[0] = v.x;
        w1[0] = v.y;
    } else if constexpr (G == 2) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p));
        w0[0] = v.x; w0[1] = v.y; w1[0] = v.z; w1[1] = v.w;
    } else {
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(p) + i);
            w0[4 * i] = v.x; w0[4 * i + 1] = v.y; w0[4 * i + 2] = v.z; w0[4 * i + 3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(p) + G / 4 + i);
            w1[4 * i] = v.x; w1[4 * i + 1] = v.y; w1[4 * i + 2] = v.z; w1[4 * i + 3] = v.w;
        }
    }
}

template <typename XT, typename YT, int VG>
__device__ __forceinline__ void store_vec(YT* p, const float (&v)[VG])
{
    if constexpr (sizeof(YT) == 4) {
#pragma unroll
        for (int i = 0; i < VG / 4; ++i)
            reinterpret_cast<float4*>(p)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
        __half2 h[VG / 2];
#pragma unroll
        for (int i = 0; i < VG / 2; ++i) h[i] = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
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
    else
        *p = __float2half_rn(v);
}

template <typename XT, int G, int P, int RW, int NW, int MINB>
__global__ void __launch_bounds__(NW * 32, MINB) spconv1x1_kernel(const ConvArgs a)
{
    constexpr int T = 32 * P;                         // pixels per tile
    constexpr int SZ = (int)sizeof(XT);
    constexpr int VG = (P * SZ >= 16) ? 16 / SZ : P;  // elements per shared-memory vector load
    constexpr int NG = P / VG;                        // vector groups per lane
    constexpr int NT = NW * 32;
    constexpr int ROWB = T * SZ;                      // bytes of one staged channel row

    extern __shared__ __align__(16) unsigned char smem[];

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int tile = blockIdx.x / a.n_rg;
    const int rg = blockIdx.x - tile * a.n_rg;
    const int q0 = tile * T;
    const int stage_bytes = a.kc * ROWB;

    // ---- block rows owned by this warp ------------------------------------------------------
    int row[RW], pos[RW], endv[RW];
    {
        const int base = rg * a.rows_per_rg;
        const int lim = min(a.rows, base + a.rows_per_rg);
#pragma unroll
        for (int s = 0; s < RW; ++s) {
            const int ps = base + s * NW + warp;
            row[s] = ps < lim ? __ldg(a.row_order + ps) : -1;
            pos[s] = row[s] >= 0 ? __ldg(a.seg_ptr + (size_t)row[s] * (a.nch + 1)) : 0;
            endv[s] = pos[s];
        }
    }

    float acc[RW][G][P];
#pragma unroll
    for (int s = 0; s < RW; ++s)
#pragma unroll
        for (int j = 0; j < G; ++j)
#pragma unroll
            for (int e = 0; e < P; ++e) acc[s][j][e] = 0.0f;

    // ---- staging set-up: this thread always copies the same pixel vector of every channel ---
    const int ev = a.ld_bytes / SZ;                   // elements per staging copy
    const int vpr = T / ev;                           // copies per channel row
    const int sv = tid % vpr;
    const int sc0 = tid / vpr;
    const int scstep = NT / vpr;
    const int sq = q0 + sv * ev;
    const bool svalid = sq < a.q_total;
    const unsigned char* ssrc = nullptr;
    if (svalid) {
        const int n = sq / a.hw;
        const int p = sq - n * a.hw;
        ssrc = static_cast<const unsigned char*>(a.x) + ((size_t)n * a.cin * a.hw + p) * SZ;
    }
    const size_t ch_bytes = (size_t)a.hw * SZ;
    const uint32_t smem_u32 = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t sdst0 = smem_u32 + sv * a.ld_bytes;

    auto stage_chunk = [&](int k) {
        if (k < a.nch && svalid) {
            const int cbase = k * a.kc;
            const int nrows = min(a.kc, a.cin - cbase);
            const uint32_t dst = sdst0 + (k % a.stages) * stage_bytes;
            const unsigned char* src = ssrc + (size_t)cbase * ch_bytes;
            if (a.ld_bytes == 16) {
                for (int c = sc0; c < nrows; c += scstep) cp_async_16(dst + c * ROWB, src + c * ch_bytes);
            } else if (a.ld_bytes == 8) {
                for (int c = sc0; c < nrows; c += scstep) cp_async_8(dst + c * ROWB, src + c * ch_bytes);
            } else if (a.ld_bytes == 4) {
                for (int c = sc0; c < nrows; c += scstep) cp_async_4(dst + c * ROWB, src + c * ch_bytes);
            } else {  // 2-byte elements at odd alignment: plain loads and shared-memory stores
                unsigned char* d = smem + (k % a.stages) * stage_bytes + sv * a.ld_bytes;
                for (int c = sc0; c < nrows; c += scstep)
                    *reinterpret_cast<unsigned short*>(d + c * ROWB) =
                        __ldg(reinterpret_cast<const unsigned short*>(src + c * ch_bytes));
            }
        }
        cp_async_commit();
    };

    for (int k = 0; k < a.stages - 1; ++k) stage_chunk(k);

    const unsigned char* xlane = smem + lane * (VG * SZ);

    // ---- main loop over channel chunks ------------------------------------------------------
    for (int k = 0; k < a.nch; ++k) {
#pragma unroll
        for (int s = 0; s < RW; ++s)
            if (row[s] >= 0) endv[s] = __ldg(a.seg_ptr + (size_t)row[s] * (a.nch + 1) + k + 1);

        if (a.stages == 2) cp_async_wait<0>();
        else if (a.stages == 3) cp_async_wait<1>();
        else cp_async_wait<2>();
        __syncthreads();          // chunk k visible to all; everyone is done with chunk k-1
        stage_chunk(k + a.stages - 1);

        const unsigned char* xs = xlane + (k % a.stages) * stage_bytes;
#pragma unroll
        for (int s = 0; s < RW; ++s) {
            if (row[s] < 0) continue;
            const int e = endv[s];
#pragma unroll 2
            for (int b = pos[s]; b < e; b += 2) {
                const int2 cc = __ldg(reinterpret_cast<const int2*>(a.cols + b));
                float w0[G], w1[G];
                load_w2<G>(a.vals + (size_t)b * G, w0, w1);
                const unsigned char* x0p = xs + cc.x * ROWB;
                const unsigned char* x1p = xs + cc.y * ROWB;
#pragma unroll
                for (int gi = 0; gi < NG; ++gi) {
                    float xv[VG];
                    XVec<XT, VG>::load(x0p + gi * (32 * VG * SZ), xv);
#pragma unroll
                    for (int j = 0; j < G; ++j)
#pragma unroll
                        for (int t = 0; t < VG; ++t)
                            acc[s][j][gi * VG + t] = fmaf(w0[j], xv[t], acc[s][j][gi * VG + t]);
                }
#pragma unroll
                for (int gi = 0; gi < NG; ++gi) {
                    float xv[VG];
                    XVec<XT, VG>::load(x1p + gi * (32 * VG * SZ), xv);
#pragma unroll
                    for (int j = 0; j < G; ++j)
#pragma unroll
                        for (int t = 0; t < VG; ++t)
                            acc[s][j][gi * VG + t] = fmaf(w1[j], xv[t], acc[s][j][gi * VG + t]);
                }
            }
            pos[s] = e;
        }
    }
    cp_async_wait<0>();

    // ---- epilogue: bias, ReLU, store --------------------------------------------------------
    auto epilogue = [&](auto* ybase) {
        using YT = std::remove_pointer_t<decltype(ybase)>;
        size_t yoff[NG];
        bool yok[NG];
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) {
            const int q = q0 + gi * (32 * VG) + lane * VG;
            yok[gi] = q < a.q_total;
            const int n = q / a.hw;
            yoff[gi] = (size_t)n * a.cout * a.hw + (q - n * a.hw);
        }
#pragma unroll
        for (int s = 0; s < RW; ++s) {
            if (row[s] < 0) continue;
#pragma unroll
            for (int j = 0; j < G; ++j) {
                const int co = row[s] * G + j;
                if (co >= a.cout) continue;
                const float bv = a.bias ? __ldg(a.bias + co) : 0.0f;
#pragma unroll
                for (int gi = 0; gi < NG; ++gi) {
                    float v[VG];
#pragma unroll
                    for (int t = 0; t < VG; ++t) {
                        v[t] = acc[s][j][gi * VG + t] + bv;
                        if (a.relu) v[t] = fmaxf(v[t], 0.0f);
                    }
                    if (a.st_vec) {
                        if (yok[gi]) store_vec<XT, YT, VG>(ybase + yoff[gi] + (size_t)co * a.hw, v);
                    } else {
#pragma unroll
                        for (int t = 0; t < VG; ++t) {
                            const int q = q0 + gi * (32 * VG) + lane * VG + t;
                            if (q < a.q_total) {
                                const int n = q / a.hw;
                                store_one<YT>(ybase + ((size_t)n * a.cout + co) * a.hw + (q - n * a.hw), v[t]);
                            }
                        }
                    }
                }
            }
        }
    };
    if constexpr (sizeof(XT) == 4) {
        epilogue(static_cast<float*>(a.y));
    } else {
        if (a.y_f32) epilogue(static_cast<float*>(a.y));
        else epilogue(static_cast<__half*>(a.y));
    }
}

// One entry of the table of compiled kernel variants.
struct KernelVariant {
    int is_f16, g, p, rw, nw, minb;
    const void* fn;
};

#define ALCS_VARIANT(XT, ISF16, G, P, RW, NW, MINB) \
    {ISF16, G, P, RW, NW, MINB, (const void*)&spconv1x1_kernel<XT, G, P, RW, NW, MINB>}

// Defined one per translation unit, concatenated by alcs_device.cu.
const KernelVariant* variants_f32_g4(int* n);
const KernelVariant* variants_f32_other(int* n);
const KernelVariant* variants_f16(int* n);

}  // namespace alcs

#endif  // ALCS_KERNELS_CUH_
