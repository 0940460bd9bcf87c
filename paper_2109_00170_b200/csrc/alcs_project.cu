// Latency model (paper, Section 3.3) and projection with bisection (Section 3.4, Algorithm 1).
//
// Host part: the linear interpolation over a layer's measured (non-zero count, run time) pairs and
// the network sum.  Device part, the data-parallel steps of Algorithm 1: the ranking key of every
// group of g adjacent filters (its squared L2 norm), the ranking of all groups of all layers (a
// radix sort from the CUDA toolkit's CUB, a library primitive), the per-layer count of the top-N
// groups that each bisection step needs, and the final mask / projected tensor.  The bisection
// itself is a few dozen iterations of host control around the counting kernel.
#include <cuda_runtime.h>

#include <cub/device/device_radix_sort.cuh>

#include <algorithm>
#include <cstdint>
#include <vector>

#include "alcs.h"

namespace alcs {
void set_cuda_error_text(const char* s);
}

namespace {

#define ALCS_CUDA(call)                                        \
    do {                                                       \
        cudaError_t e_ = (call);                               \
        if (e_ != cudaSuccess) {                               \
            alcs::set_cuda_error_text(cudaGetErrorString(e_)); \
            (void)cudaGetLastError();                          \
            return ALCS_ERR_CUDA;                              \
        }                                                      \
    } while (0)

// Eq. for T^(s): t_1 + sum_i delta_i alpha_i min(k_{i+1} - k_i, s - k_i), evaluated term by term.
double interpolate(const alcs_latency_table& tab, int64_t s)
{
    double total = tab.t[0];
    for (int i = 0; i + 1 < tab.n_knots; ++i) {
        const double delta = s >= tab.k[i] ? 1.0 : 0.0;
        const double width = (double)tab.k[i + 1] - (double)tab.k[i];
        const double alpha = (tab.t[i + 1] - tab.t[i]) / width;
        total += delta * alpha * std::min(width, (double)s - (double)tab.k[i]);
    }
    return total;
}

int check_table(const alcs_latency_table* tab)
{
    if (!tab || tab->n_knots < 2 || !tab->k || !tab->t) return ALCS_ERR_INVALID_ARG;
    for (int i = 0; i + 1 < tab->n_knots; ++i)
        if (tab->k[i + 1] <= tab->k[i]) return ALCS_ERR_INVALID_ARG;
    return ALCS_OK;
}

// key[group] = sum over the g filters of the group of the squared element: fp32, one rounded
// multiply and one rounded add per element, filters in ascending order (no fused multiply-add, so
// that the ranking is reproducible bit for bit).  Group (r, c) of a [cout][cols] layer covers
// elements (r*g + j, c); a missing filter of a ragged last group counts as zero.  Also writes the
// identity permutation that the sort carries along.
__global__ void group_keys_kernel(const float* __restrict__ u, int cout, int cols, int g, long long base,
                                  unsigned* __restrict__ keys, unsigned* __restrict__ idx)
{
    const int rows = (cout + g - 1) / g;
    const long long n = (long long)rows * cols;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(i / cols);
        const int c = (int)(i - (long long)r * cols);
        float acc = 0.0f;
        for (int j = 0; j < g; ++j) {
            const int co = r * g + j;
            if (co >= cout) break;
            const float v = __ldg(u + (size_t)co * cols + c);
            acc = __fadd_rn(acc, __fmul_rn(v, v));
        }
        keys[base + i] = __float_as_uint(acc);      // non-negative floats order like their bit patterns
        idx[base + i] = (unsigned)(base + i);
    }
}

// layer_of[i] = layer of the i-th ranked group (binary search over the layers' group offsets)
__global__ void ranked_layer_kernel(const unsigned* __restrict__ idx, long long total, const long long* __restrict__ off,
                                    int n_layers, unsigned short* __restrict__ layer_of)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long gidx = idx[i];
        int lo = 0, hi = n_layers - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (off[mid] <= gidx) lo = mid; else hi = mid - 1;
        }
        layer_of[i] = (unsigned short)lo;
    }
}

constexpr int kMaxLayers = 4096;

// counts[l] += number of the top-n ranked groups that belong to layer l
__global__ void count_top_kernel(const unsigned short* __restrict__ layer_of, long long n, int n_layers,
                                 unsigned long long* __restrict__ counts)
{
    extern __shared__ unsigned int hist[];
    for (int i = threadIdx.x; i < n_layers; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        atomicAdd(&hist[layer_of[i]], 1u);
    __syncthreads();
    for (int i = threadIdx.x; i < n_layers; i += blockDim.x)
        if (hist[i]) atomicAdd(&counts[i], (unsigned long long)hist[i]);
}

// mask[group] = 1 for the n best-ranked groups, 0 for the others
__global__ void write_mask_kernel(const unsigned* __restrict__ idx, long long total, long long n, uint8_t* __restrict__ mask)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
        mask[idx[i]] = i < n ? 1 : 0;
}

// u_out = u where the element's group is kept, +0 elsewhere
__global__ void apply_mask_kernel(const float* __restrict__ u, const uint8_t* __restrict__ mask, int cout, int cols, int g,
                                  float* __restrict__ out)
{
    const long long n = (long long)cout * cols;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int co = (int)(i / cols);
        const int c = (int)(i - (long long)co * cols);
        out[i] = mask[(size_t)(co / g) * cols + c] ? u[i] : 0.0f;
    }
}

unsigned blocks_for(long long n, int threads = 256)
{
    return (unsigned)std::max<long long>(1, std::min<long long>((n + threads - 1) / threads, 148 * 16));
}

struct DeviceBuffers {
    void* p[8] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    ~DeviceBuffers() { for (void* q : p) if (q) cudaFree(q); }
};

}  // namespace

extern "C" {

ALCS_API int alcs_layer_latency(const alcs_latency_table* tab, int64_t s, double* out)
{
    if (!out) return ALCS_ERR_INVALID_ARG;
    const int rc = check_table(tab);
    if (rc) return rc;
    *out = interpolate(*tab, s);
    return ALCS_OK;
}

ALCS_API int alcs_network_latency(double tau, const alcs_latency_table* tabs, int n_layers, const int64_t* s, double* out)
{
    if (!out || n_layers < 0 || (n_layers && (!tabs || !s))) return ALCS_ERR_INVALID_ARG;
    double total = tau;
    for (int l = 0; l < n_layers; ++l) {
        const int rc = check_table(&tabs[l]);
        if (rc) return rc;
        total += interpolate(tabs[l], s[l]);
    }
    *out = total;
    return ALCS_OK;
}

ALCS_API int alcs_project_bisection(const float* const* u_tilde, const int* cout, const int* cols, int n_layers, int g,
                                    const alcs_latency_table* tabs, double tau, double t_budget, double eps,
                                    uint8_t* mask_out, float* const* u_out, int64_t* kept_per_layer,
                                    alcs_projection_result* result, void* cuda_stream)
{
    if (!u_tilde || !cout || !cols || !tabs || !mask_out || n_layers <= 0 || g < 1 || g > 64) return ALCS_ERR_INVALID_ARG;
    if (n_layers > kMaxLayers) return ALCS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    std::vector<long long> off(n_layers + 1, 0);
    for (int l = 0; l < n_layers; ++l) {
        if (!u_tilde[l] || cout[l] <= 0 || cols[l] <= 0) return ALCS_ERR_INVALID_ARG;
        const int rc = check_table(&tabs[l]);
        if (rc) return rc;
        off[l + 1] = off[l] + (long long)((cout[l] + g - 1) / g) * cols[l];
    }
    const long long total = off[n_layers];
    if (total >= (1ll << 32)) return ALCS_ERR_SHAPE;        // group indices are 32-bit

    DeviceBuffers b;
    unsigned *keys = nullptr, *idx = nullptr, *keys2 = nullptr, *idx2 = nullptr;
    unsigned short* layer_of = nullptr;
    long long* d_off = nullptr;
    unsigned long long* d_counts = nullptr;
    auto alloc = [&](int slot, size_t bytes) { return cudaMalloc(&b.p[slot], std::max<size_t>(bytes, 16)); };
    if (alloc(0, total * 4) || alloc(1, total * 4) || alloc(2, total * 4) || alloc(3, total * 4) || alloc(4, total * 2) ||
        alloc(5, (n_layers + 1) * 8) || alloc(6, n_layers * 8)) {
        (void)cudaGetLastError();
        return ALCS_ERR_ALLOC;
    }
    keys = (unsigned*)b.p[0]; idx = (unsigned*)b.p[1]; keys2 = (unsigned*)b.p[2]; idx2 = (unsigned*)b.p[3];
    layer_of = (unsigned short*)b.p[4]; d_off = (long long*)b.p[5]; d_counts = (unsigned long long*)b.p[6];

    // steps 1-2: group keys, then rank all groups of all layers, largest key first.  The radix sort
    // is stable, so equal keys stay in (layer, group) order.
    for (int l = 0; l < n_layers; ++l) {
        const long long n = off[l + 1] - off[l];
        group_keys_kernel<<<blocks_for(n), 256, 0, st>>>(u_tilde[l], cout[l], cols[l], g, off[l], keys, idx);
    }
    ALCS_CUDA(cudaGetLastError());
    size_t tmp_bytes = 0;
    ALCS_CUDA(cub::DeviceRadixSort::SortPairsDescending(nullptr, tmp_bytes, keys, keys2, idx, idx2, (int)total, 0, 32, st));
    if (cudaMalloc(&b.p[7], std::max<size_t>(tmp_bytes, 16)) != cudaSuccess) {
        (void)cudaGetLastError();
        return ALCS_ERR_ALLOC;
    }
    ALCS_CUDA(cub::DeviceRadixSort::SortPairsDescending(b.p[7], tmp_bytes, keys, keys2, idx, idx2, (int)total, 0, 32, st));
    ALCS_CUDA(cudaMemcpyAsync(d_off, off.data(), (n_layers + 1) * 8, cudaMemcpyHostToDevice, st));
    ranked_layer_kernel<<<blocks_for(total), 256, 0, st>>>(idx2, total, d_off, n_layers, layer_of);
    ALCS_CUDA(cudaGetLastError());

    // T(U) for "the top-n groups kept": per-layer counts on the device, the interpolation on the host
    std::vector<unsigned long long> counts(n_layers);
    std::vector<int64_t> nz(n_layers);
    auto latency_of_top = [&](long long n, double* t) -> int {
        ALCS_CUDA(cudaMemsetAsync(d_counts, 0, n_layers * 8, st));
        if (n > 0) count_top_kernel<<<blocks_for(n), 256, n_layers * 4, st>>>(layer_of, n, n_layers, d_counts);
        ALCS_CUDA(cudaGetLastError());
        ALCS_CUDA(cudaMemcpyAsync(counts.data(), d_counts, n_layers * 8, cudaMemcpyDeviceToHost, st));
        ALCS_CUDA(cudaStreamSynchronize(st));
        for (int l = 0; l < n_layers; ++l) nz[l] = (int64_t)counts[l] * g;
        double total_t = tau;
        for (int l = 0; l < n_layers; ++l) total_t += interpolate(tabs[l], nz[l]);
        *t = total_t;
        return ALCS_OK;
    };

    // steps 3-15 of Algorithm 1
    long long n0 = 0, n1 = total;
    double t0 = 0, t1 = 0;
    int rc = latency_of_top(0, &t0);
    if (rc) return rc;
    rc = latency_of_top(total, &t1);
    if (rc) return rc;
    int iters = 0;
    while (t1 - t0 > eps && n1 - n0 > 1) {      // the second test ends a bracket that cannot shrink
        const long long n = (n0 + n1) / 2;
        double t = 0;
        rc = latency_of_top(n, &t);
        if (rc) return rc;
        if (t < t_budget) { t0 = t; n0 = n; } else { t1 = t; n1 = n; }
        ++iters;
    }
    const long long n_keep = (n0 + n1) / 2;
    double t_final = 0;
    rc = latency_of_top(n_keep, &t_final);
    if (rc) return rc;

    write_mask_kernel<<<blocks_for(total), 256, 0, st>>>(idx2, total, n_keep, mask_out);
    ALCS_CUDA(cudaGetLastError());
    if (u_out) {
        for (int l = 0; l < n_layers; ++l) {
            if (!u_out[l]) continue;
            apply_mask_kernel<<<blocks_for((long long)cout[l] * cols[l]), 256, 0, st>>>(u_tilde[l], mask_out + off[l], cout[l], cols[l], g, u_out[l]);
        }
        ALCS_CUDA(cudaGetLastError());
    }
    ALCS_CUDA(cudaStreamSynchronize(st));       // the temporaries are freed on return
    if (kept_per_layer)
        for (int l = 0; l < n_layers; ++l) kept_per_layer[l] = (int64_t)counts[l];
    if (result) {
        result->n_keep = n_keep; result->n0 = n0; result->n1 = n1; result->iters = iters; result->latency = t_final;
        result->n_groups = total;
    }
    return ALCS_OK;
}

}  // extern "C"
