// Latency model (paper, Section 3.3) and projection with bisection (Section 3.4, Algorithm 1).
//
// Host part: the linear interpolation over a layer's measured (non-zero count, run time) pairs and
// the network sum.  Device part, the data-parallel steps of Algorithm 1: the ranking key of every
// group of g adjacent filters (its squared L2 norm), the ranking of all groups of all layers (a
// radix sort from the CUDA toolkit's CUB, a library primitive), the layer of every ranked group with
// per-bucket layer histograms, and the final mask / projected tensor.  The search over the length of
// the kept prefix of the ranked list runs on the host from one copy of those two arrays.
#include <cuda_runtime.h>

#include <cub/device/device_radix_sort.cuh>

#include <algorithm>
#include <cstdint>
#include <mutex>
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

constexpr long long kRankBucket = 4096;

// page-locked host staging area of alcs_project_bisection, shared by all calls (one call at a time uses it)
std::mutex g_staging_mu;
void* g_staging = nullptr;
size_t g_staging_bytes = 0;

// hist[b][l] = how many of the ranked entries b*kRankBucket .. (b+1)*kRankBucket - 1 belong to layer l
// (one thread block per bucket, a shared-memory histogram)
__global__ void bucket_histogram_kernel(const unsigned short* __restrict__ layer_of, long long total, int n_layers,
                                        unsigned* __restrict__ hist)
{
    extern __shared__ unsigned int h[];
    for (int i = threadIdx.x; i < n_layers; i += blockDim.x) h[i] = 0;
    __syncthreads();
    const long long b0 = (long long)blockIdx.x * kRankBucket;
    const long long b1 = b0 + kRankBucket < total ? b0 + kRankBucket : total;
    for (long long i = b0 + threadIdx.x; i < b1; i += blockDim.x) atomicAdd(&h[layer_of[i]], 1u);
    __syncthreads();
    for (int i = threadIdx.x; i < n_layers; i += blockDim.x) hist[(size_t)blockIdx.x * n_layers + i] = h[i];
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
    if (total >= (1ll << 31)) return ALCS_ERR_SHAPE;        // the sort takes a 32-bit signed item count
    int dev = 0, sms = 0;
    ALCS_CUDA(cudaGetDevice(&dev));
    ALCS_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    auto blocks_for = [&](long long n) {
        return (unsigned)std::max<long long>(1, std::min<long long>((n + 255) / 256, (long long)sms * 16));
    };

    // One stream-ordered allocation for everything: after the first call the memory comes back from
    // the runtime's pool without touching the driver.
    const long long n_buckets = (total + kRankBucket - 1) / kRankBucket;
    size_t sort_bytes = 0;
    ALCS_CUDA(cub::DeviceRadixSort::SortPairsDescending(nullptr, sort_bytes, (unsigned*)nullptr, (unsigned*)nullptr,
                                                       (unsigned*)nullptr, (unsigned*)nullptr, (int)total, 0, 32, st));
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t b_keys = up((size_t)total * 4), b_lay = up((size_t)total * 2), b_off = up((size_t)(n_layers + 1) * 8);
    const size_t b_hist = up((size_t)std::max<long long>(n_buckets, 1) * n_layers * 4);
    const size_t bytes = 4 * b_keys + b_lay + b_off + b_hist + up(sort_bytes) + 256;
    unsigned char* pool = nullptr;
    if (cudaMallocAsync(&pool, bytes, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return ALCS_ERR_ALLOC;
    }
    struct Release {
        unsigned char* p; cudaStream_t s;
        ~Release() { cudaFreeAsync(p, s); }
    } release{pool, st};
    unsigned* keys = (unsigned*)pool;
    unsigned* idx = (unsigned*)(pool + b_keys);
    unsigned* keys2 = (unsigned*)(pool + 2 * b_keys);
    unsigned* idx2 = (unsigned*)(pool + 3 * b_keys);
    unsigned short* layer_of = (unsigned short*)(pool + 4 * b_keys);
    long long* d_off = (long long*)(pool + 4 * b_keys + b_lay);
    unsigned* d_hist = (unsigned*)(pool + 4 * b_keys + b_lay + b_off);
    void* sort_tmp = pool + 4 * b_keys + b_lay + b_off + b_hist;

    // Ranking (Algorithm 1: the groups of all layers sorted together by norm, largest first).  The radix
    // sort is stable, so equal keys stay in (layer, group) order.  Then, for the ranked list, the layer
    // of every entry and, per bucket of kRankBucket consecutive ranks, how many entries each layer has.
    for (int l = 0; l < n_layers; ++l) {
        const long long n = off[l + 1] - off[l];
        group_keys_kernel<<<blocks_for(n), 256, 0, st>>>(u_tilde[l], cout[l], cols[l], g, off[l], keys, idx);
    }
    ALCS_CUDA(cudaGetLastError());
    ALCS_CUDA(cub::DeviceRadixSort::SortPairsDescending(sort_tmp, sort_bytes, keys, keys2, idx, idx2, (int)total, 0, 32, st));
    ALCS_CUDA(cudaMemcpyAsync(d_off, off.data(), (n_layers + 1) * 8, cudaMemcpyHostToDevice, st));
    ranked_layer_kernel<<<blocks_for(total), 256, 0, st>>>(idx2, total, d_off, n_layers, layer_of);
    ALCS_CUDA(cudaGetLastError());
    if (n_buckets > 0) {
        bucket_histogram_kernel<<<(unsigned)n_buckets, 256, n_layers * 4, st>>>(layer_of, total, n_layers, d_hist);
        ALCS_CUDA(cudaGetLastError());
    }

    // The latency of "the N best-ranked groups kept" depends on N only through the number of kept
    // groups per layer, a monotone step function of N.  One copy brings what is needed to evaluate it
    // for any N on the host: the bucket histograms (turned into prefix counts) and the ranked list's
    // layers, of which at most one bucket is scanned per evaluation.  No device work per search step.
    // (page-locked staging memory, kept between calls: a copy into pageable memory is several times slower)
    const size_t hist_bytes = (size_t)n_buckets * n_layers * 4, lay_bytes = (size_t)total * 2;
    std::unique_lock<std::mutex> staging_lock(g_staging_mu);
    if (g_staging_bytes < up(hist_bytes) + lay_bytes + 16) {
        if (g_staging) cudaFreeHost(g_staging);
        g_staging = nullptr;
        g_staging_bytes = 0;
        const size_t want = (up(hist_bytes) + lay_bytes + 16) * 5 / 4;
        if (cudaMallocHost(&g_staging, want) != cudaSuccess) {
            (void)cudaGetLastError();
            return ALCS_ERR_ALLOC;
        }
        g_staging_bytes = want;
    }
    const unsigned* hist = reinterpret_cast<const unsigned*>(g_staging);
    const unsigned short* lay = reinterpret_cast<const unsigned short*>(static_cast<unsigned char*>(g_staging) + up(hist_bytes));
    if (total > 0) {
        ALCS_CUDA(cudaMemcpyAsync(g_staging, d_hist, hist_bytes, cudaMemcpyDeviceToHost, st));
        ALCS_CUDA(cudaMemcpyAsync(static_cast<unsigned char*>(g_staging) + up(hist_bytes), layer_of, lay_bytes, cudaMemcpyDeviceToHost, st));
    }
    ALCS_CUDA(cudaStreamSynchronize(st));
    std::vector<long long> prefix((size_t)(n_buckets + 1) * n_layers, 0);     // groups of layer l among ranks < b*kRankBucket
    for (long long bk = 0; bk < n_buckets; ++bk)
        for (int l = 0; l < n_layers; ++l)
            prefix[(size_t)(bk + 1) * n_layers + l] = prefix[(size_t)bk * n_layers + l] + hist[(size_t)bk * n_layers + l];
    std::vector<long long> counts(n_layers);
    auto latency_of_top = [&](long long n) {
        const long long bk = n / kRankBucket;
        for (int l = 0; l < n_layers; ++l) counts[l] = prefix[(size_t)bk * n_layers + l];
        for (long long i = bk * kRankBucket; i < n; ++i) ++counts[lay[(size_t)i]];
        double t = tau;
        for (int l = 0; l < n_layers; ++l) t += interpolate(tabs[l], (int64_t)counts[l] * g);
        return t;
    };

    // Search: the bracket [lo, hi] of prefix lengths always has latency(lo) on the budget's near side
    // as far as it is known and is halved until the latencies of its two ends are within eps of each
    // other (Section 3.4, Algorithm 1); a bracket of width 1 cannot shrink further and also ends it.
    long long lo = 0, hi = total;
    double t_lo = latency_of_top(lo), t_hi = latency_of_top(hi);
    int iters = 0;
    while (t_hi - t_lo > eps && hi - lo > 1) {
        const long long mid = (lo + hi) / 2;
        const double t = latency_of_top(mid);
        if (t < t_budget) { t_lo = t; lo = mid; } else { t_hi = t; hi = mid; }
        ++iters;
    }
    const long long n_keep = (lo + hi) / 2;
    const double t_final = latency_of_top(n_keep);      // (leaves the kept counts of the result in `counts`)

    write_mask_kernel<<<blocks_for(total), 256, 0, st>>>(idx2, total, n_keep, mask_out);
    ALCS_CUDA(cudaGetLastError());
    if (u_out) {
        for (int l = 0; l < n_layers; ++l) {
            if (!u_out[l]) continue;
            apply_mask_kernel<<<blocks_for((long long)cout[l] * cols[l]), 256, 0, st>>>(u_tilde[l], mask_out + off[l], cout[l], cols[l], g, u_out[l]);
        }
        ALCS_CUDA(cudaGetLastError());
    }
    ALCS_CUDA(cudaStreamSynchronize(st));
    if (kept_per_layer)
        for (int l = 0; l < n_layers; ++l) kept_per_layer[l] = (int64_t)counts[l];
    if (result) {
        result->n_keep = n_keep; result->n0 = lo; result->n1 = hi; result->iters = iters; result->latency = t_final;
        result->n_groups = total;
    }
    return ALCS_OK;
}

}  // extern "C"
