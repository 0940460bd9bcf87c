// Compiled variants of the general k x k sparse convolution kernel (fp32) and their launcher.
#include "alcs_conv2d.cuh"

#include <mutex>

namespace alcs {

namespace {

struct Conv2dVariant {
    int g, p, st, ni;
    const void* fn[2];      // [0] all channels in one chunk, [1] chunked
    bool ready[2];
};

#define ALCS_C2D_N(G, P, ST, NI)                                                            \
    {G, P, ST, NI, {(const void*)&spconv2d_kernel<G, P, ST, kConv2dWarps, false, NI>,       \
                    (const void*)&spconv2d_kernel<G, P, ST, kConv2dWarps, true, NI>}, {false, false}}
#define ALCS_C2D(G, P, ST) ALCS_C2D_N(G, P, ST, 1)
#define ALCS_C2D_G(G)                                                                                      \
    ALCS_C2D(G, 2, 1), ALCS_C2D(G, 4, 1), ALCS_C2D(G, 8, 1), ALCS_C2D(G, 2, 2), ALCS_C2D(G, 4, 2), ALCS_C2D(G, 8, 2), \
    ALCS_C2D_N(G, 4, 1, 2), ALCS_C2D_N(G, 8, 1, 2), ALCS_C2D_N(G, 8, 1, 4), ALCS_C2D_N(G, 4, 2, 2), ALCS_C2D_N(G, 8, 2, 2), \
    ALCS_C2D_N(G, 8, 2, 4)

// (g = 16 with 8 positions per lane would need 128 accumulator registers: left out)
Conv2dVariant kTable[] = {ALCS_C2D_G(1), ALCS_C2D_G(2), ALCS_C2D_G(4), ALCS_C2D_G(8),
                          ALCS_C2D(16, 2, 1), ALCS_C2D(16, 4, 1), ALCS_C2D(16, 2, 2), ALCS_C2D(16, 4, 2),
                          ALCS_C2D_N(16, 4, 1, 2), ALCS_C2D_N(16, 4, 2, 2)};
std::mutex g_c2d_mu;

Conv2dVariant* find(int g, int p, int st, int ni)
{
    for (auto& v : kTable)
        if (v.g == g && v.p == p && v.st == st && v.ni == ni) return &v;
    return nullptr;
}

}  // namespace

bool conv2d_variant_exists(int g, int p, int stride, int ni) { return find(g, p, stride, ni) != nullptr; }

cudaError_t launch_conv2d(int g, int p, int stride, int ni, const Conv2dArgs& a, unsigned grid, size_t smem, cudaStream_t st)
{
    Conv2dVariant* v = find(g, p, stride, ni);
    if (!v) return cudaErrorInvalidValue;
    const int ch = a.nch > 1 ? 1 : 0;
    {
        std::lock_guard<std::mutex> lk(g_c2d_mu);
        if (!v->ready[ch]) {
            cudaError_t e = cudaFuncSetAttribute(v->fn[ch], cudaFuncAttributeMaxDynamicSharedMemorySize, kConv2dMaxDynSmem);
            if (e != cudaSuccess) return e;
            v->ready[ch] = true;
        }
    }
    Conv2dArgs args = a;
    void* params[] = {&args};
    return cudaLaunchKernel(v->fn[ch], dim3(grid), dim3(kConv2dWarps * 32), params, smem, st);
}

}  // namespace alcs
