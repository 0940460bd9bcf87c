// Small-problem kernel of the sparse pointwise convolution (fp32): no shared-memory staging of X.
//
// At batch 1 (the paper's own latency setting) a layer is a few hundred kilobytes of X and a few
// megaflops: the time goes to latency, not to bandwidth or arithmetic.  The staged kernel makes every
// thread block copy all input channels of its pixel tile through the ring, chunk after chunk, before
// its last multiply can start.  Here a thread block is one (block row, image, pixel tile); its KS
// warps split the row's kept columns among themselves (warp k takes blocks k, k+KS, ...), read the
// input vectors those columns address straight from global memory (the loop of Section 3.2.2,
// "Efficient multiplication computation", as printed: load the column's g weights, load the input
// vector at the column offset, multiply-accumulate), with several blocks' loads in flight, and the
// partial sums are added up through shared memory in a fixed order (warp 0, 1, ...: deterministic).
// It walks the canonical storage format (row_ptr / col_idx / vals), not a launch schedule.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "alcs_gather.h"

namespace alcs {

namespace {

constexpr int kUnroll = 4;      // blocks whose loads are issued together

template <int G>
__device__ __forceinline__ void load_weights(const float* __restrict__ p, float (&w)[G])
{
    if constexpr (G % 4 == 0) {
#pragma unroll
        for (int i = 0; i < G / 4; ++i) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(p) + i);
            w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
        }
    } else if constexpr (G == 2) {
        const float2 v = __ldg(reinterpret_cast<const float2*>(p));
        w[0] = v.x; w[1] = v.y;
    } else {
#pragma unroll
        for (int i = 0; i < G; ++i) w[i] = __ldg(p + i);
    }
}

// VEC: rows of X are 16-byte aligned multiples of 4 pixels; a lane then owns pixels
// t0 + 4*lane + 128*i + (0..3) and reads them as one 128-bit load.  Otherwise a lane owns pixels
// t0 + lane + 32*i and reads them one by one.
template <int G, int P, bool VEC>
__global__ void __launch_bounds__(512) gather_kernel(const GatherArgs a)
{
    extern __shared__ __align__(16) float red[];         // [KS][G*P][32]
    const int lane = threadIdx.x & 31;
    const int ks = threadIdx.x >> 5;
    const int KS = blockDim.x >> 5;
    const int tile = blockIdx.x % a.tiles;
    const int img = (blockIdx.x / a.tiles) % a.n;
    const int r = blockIdx.x / (a.tiles * a.n);
    const int t0 = tile * (32 * P);

    int pix[P];                                          // pixel of each accumulator column, or -1
#pragma unroll
    for (int i = 0; i < P; ++i) {
        const int p = VEC ? t0 + 4 * lane + 128 * (i / 4) + (i % 4) : t0 + lane + 32 * i;
        pix[i] = p < a.hw ? p : -1;
    }
    float acc[G][P];
#pragma unroll
    for (int j = 0; j < G; ++j)
#pragma unroll
        for (int i = 0; i < P; ++i) acc[j][i] = 0.0f;

    const float* ximg = a.x + (size_t)img * a.cin * a.hw;
    // Programmatic dependent launch: the next kernel on the stream may start its own set-up now; this
    // kernel reads what does not depend on its predecessor (the row's column indices and weights,
    // pulled towards the SM here) and only then waits for the predecessor, whose output is its x.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int k_first = __ldg(a.row_ptr + r);
    const int k1 = __ldg(a.row_ptr + r + 1);
    // Rows that fit are copied into shared memory (the area the partial sums use later) before the wait, so
    // that afterwards only the input vectors remain to be fetched: one memory round trip per batch of blocks
    // instead of two dependent ones (column index, then the input it addresses).
    const bool staged = a.stage_blocks > 0 && k1 - k_first <= a.stage_blocks;
    int* scol = reinterpret_cast<int*>(red);                         // [stage_blocks]
    float* sval = red + ((a.stage_blocks + 3) & ~3);                 // [stage_blocks][G], 16-byte aligned
    if (staged) {
        const int nbk = k1 - k_first;
        for (int i = threadIdx.x; i < nbk; i += blockDim.x) scol[i] = __ldg(a.col_idx + k_first + i);
        const float* vsrc = a.vals + (size_t)k_first * G;
        if constexpr (G % 4 == 0) {
            for (int i = threadIdx.x; i < nbk * (G / 4); i += blockDim.x)
                reinterpret_cast<float4*>(sval)[i] = __ldg(reinterpret_cast<const float4*>(vsrc) + i);
        } else {
            for (int i = threadIdx.x; i < nbk * G; i += blockDim.x) sval[i] = __ldg(vsrc + i);
        }
        __syncthreads();
    } else {
        const char* cb = reinterpret_cast<const char*>(a.col_idx + k_first);
        const char* vb = reinterpret_cast<const char*>(a.vals + (size_t)k_first * G);
        const long long cbytes = (long long)(k1 - k_first) * 4, vbytes = cbytes * G;
        for (long long o = (long long)threadIdx.x * 128; o < cbytes; o += (long long)blockDim.x * 128)
            asm volatile("prefetch.global.L2 [%0];\n" ::"l"(cb + o));
        for (long long o = (long long)threadIdx.x * 128; o < vbytes; o += (long long)blockDim.x * 128)
            asm volatile("prefetch.global.L2 [%0];\n" ::"l"(vb + o));
    }
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    for (int k = k_first + ks; k < k1; k += KS * kUnroll) {
        float w[kUnroll][G];
        float xv[kUnroll][P];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int kk = k + u * KS;
            const bool on = kk < k1;
            const int col = on ? (staged ? scol[kk - k_first] : __ldg(a.col_idx + kk)) : 0;
            if (on && staged) {
                if constexpr (G % 4 == 0) {
#pragma unroll
                    for (int i = 0; i < G / 4; ++i) {
                        const float4 v = reinterpret_cast<const float4*>(sval)[(kk - k_first) * (G / 4) + i];
                        w[u][4 * i] = v.x; w[u][4 * i + 1] = v.y; w[u][4 * i + 2] = v.z; w[u][4 * i + 3] = v.w;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < G; ++j) w[u][j] = sval[(kk - k_first) * G + j];
                }
            } else if (on) {
                load_weights<G>(a.vals + (size_t)kk * G, w[u]);
            } else {
#pragma unroll
                for (int j = 0; j < G; ++j) w[u][j] = 0.0f;
            }
            const float* xr = ximg + (size_t)col * a.hw;
            if constexpr (VEC) {
#pragma unroll
                for (int i = 0; i < P; i += 4) {
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (on && pix[i] >= 0) v = __ldg(reinterpret_cast<const float4*>(xr + pix[i]));
                    xv[u][i] = v.x; xv[u][i + 1] = v.y; xv[u][i + 2] = v.z; xv[u][i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < P; ++i) xv[u][i] = (on && pix[i] >= 0) ? __ldg(xr + pix[i]) : 0.0f;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
#pragma unroll
            for (int j = 0; j < G; ++j)
#pragma unroll
                for (int i = 0; i < P; ++i) acc[j][i] = fmaf(w[u][j], xv[u][i], acc[j][i]);
    }

    // add the warps' partial sums in warp order, then bias, ReLU, store
    if (staged) __syncthreads();        // (the staged row shares the area of the partial sums)
#pragma unroll
    for (int j = 0; j < G; ++j)
#pragma unroll
        for (int i = 0; i < P; ++i) red[(ks * (G * P) + j * P + i) * 32 + lane] = acc[j][i];
    __syncthreads();
    float* yimg = a.y + (size_t)img * a.cout * a.hw;
    for (int e = ks; e < G * P; e += KS) {
        const int j = e / P, i = e - j * P;
        float s = 0.0f;
        for (int q = 0; q < KS; ++q) s += red[(q * (G * P) + e) * 32 + lane];
        const int co = r * G + j;
        const int p = VEC ? t0 + 4 * lane + 128 * (i / 4) + (i % 4) : t0 + lane + 32 * i;
        if (co < a.cout && p < a.hw) {
            s += a.bias ? __ldg(a.bias + co) : 0.0f;
            if (a.relu) s = fmaxf(s, 0.0f);
            yimg[(size_t)co * a.hw + p] = s;
        }
    }
}

template <int G, int P>
cudaError_t launch_gp(const GatherArgs& a, bool vec, unsigned grid, int ks, cudaStream_t st)
{
    const size_t red_bytes = (size_t)ks * G * P * 32 * sizeof(float);
    const size_t smem = std::max(red_bytes, (size_t)a.stage_blocks * 4 * (G + 1) + 16);
    // launched so that it may overlap the tail of the kernel before it on the stream (it waits for that
    // kernel before it touches x or y); a CUDA graph keeps the same programmatic edge
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(ks * 32);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    GatherArgs args = a;
    void* params[] = {&args};
    const void* fn = vec ? (const void*)&gather_kernel<G, P, true> : (const void*)&gather_kernel<G, P, false>;
    return cudaLaunchKernelExC(&lc, fn, params);
}

template <int G>
cudaError_t launch_g(const GatherArgs& a, int p, bool vec, unsigned grid, int ks, cudaStream_t st)
{
    if constexpr (G <= 4) {
        if (p == 8) return launch_gp<G, 8>(a, vec, grid, ks, st);
    }
    if constexpr (G <= 8) {
        if (p == 4) return launch_gp<G, 4>(a, vec, grid, ks, st);
    }
    if (p == 2 && !vec) return launch_gp<G, 2>(a, false, grid, ks, st);
    return cudaErrorInvalidValue;
}

}  // namespace

bool gather_config_ok(int g, int p, int ks, bool vec)
{
    if (g != 1 && g != 2 && g != 4 && g != 8 && g != 16) return false;
    if (p != 2 && p != 4 && p != 8) return false;
    if (g * p > 32) return false;            // accumulators, weights and inputs of four blocks must fit the registers
    if (p == 2 && vec) return false;
    if (ks < 1 || ks > 16) return false;
    return (size_t)ks * g * p * 32 * sizeof(float) <= 48 * 1024;
}

int gather_stage_blocks(int g, int max_row_blocks)
{
    if (max_row_blocks <= 0) return 0;
    return (size_t)max_row_blocks * 4 * (g + 1) + 16 <= 48 * 1024 ? max_row_blocks : 0;
}

cudaError_t launch_gather(int g, int p, int ks, const GatherArgs& a, cudaStream_t st)
{
    const bool vec = a.vec != 0;
    if (!gather_config_ok(g, p, ks, vec)) return cudaErrorInvalidValue;
    const long long grid = (long long)a.rows * a.n * a.tiles;
    if (grid <= 0 || grid > 0x7fffffffll) return cudaErrorInvalidValue;
    switch (g) {
        case 1: return launch_g<1>(a, p, vec, (unsigned)grid, ks, st);
        case 2: return launch_g<2>(a, p, vec, (unsigned)grid, ks, st);
        case 4: return launch_g<4>(a, p, vec, (unsigned)grid, ks, st);
        case 8: return launch_g<8>(a, p, vec, (unsigned)grid, ks, st);
        case 16: return launch_g<16>(a, p, vec, (unsigned)grid, ks, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace alcs
