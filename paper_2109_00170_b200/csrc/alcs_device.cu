// Device-facing half of libalcs: upload of the packed weights and their launch schedules, launch
// planning, the convolution entry points, the tuner, the host-buffer variant and the layer stack.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "alcs_internal.h"
#include "alcs_kernels.cuh"

namespace alcs {
void set_cuda_error_text(const char* s);
}

namespace {

using alcs::ConvArgs;
using alcs::KernelVariant;

#define ALCS_CUDA(call)                                        \
    do {                                                       \
        cudaError_t e_ = (call);                               \
        if (e_ != cudaSuccess) {                               \
            alcs::set_cuda_error_text(cudaGetErrorString(e_)); \
            (void)cudaGetLastError();                          \
            return ALCS_ERR_CUDA;                              \
        }                                                      \
    } while (0)

constexpr int kMaxSmem = 227 * 1024;

struct VariantInfo {
    KernelVariant v;
    int regs = 0;
    bool ready = false;
};

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
    bool ok = false;
};

std::mutex g_mu;
std::vector<VariantInfo> g_variants;
DeviceInfo g_dev[64];

void init_variants_locked()
{
    if (!g_variants.empty()) return;
    int n = 0;
    const KernelVariant* t = alcs::variants_f32_g4(&n);
    for (int i = 0; i < n; ++i) g_variants.push_back({t[i]});
    t = alcs::variants_f32_other(&n);
    for (int i = 0; i < n; ++i) g_variants.push_back({t[i]});
    t = alcs::variants_f16(&n);
    for (int i = 0; i < n; ++i) g_variants.push_back({t[i]});
}

int device_info(int dev, DeviceInfo* out)
{
    if (dev < 0 || dev >= 64) return ALCS_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_dev[dev].ok) {
        ALCS_CUDA(cudaDeviceGetAttribute(&g_dev[dev].sms, cudaDevAttrMultiProcessorCount, dev));
        ALCS_CUDA(cudaDeviceGetAttribute(&g_dev[dev].smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        g_dev[dev].ok = true;
    }
    *out = g_dev[dev];
    return ALCS_OK;
}

// Make a variant launchable with large dynamic shared memory (once per process).
int prepare_variant(VariantInfo& vi)
{
    std::lock_guard<std::mutex> lk(g_mu);
    if (vi.ready) return ALCS_OK;
    ALCS_CUDA(cudaFuncSetAttribute(vi.v.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
    cudaFuncAttributes fa;
    ALCS_CUDA(cudaFuncGetAttributes(&fa, vi.v.fn));
    vi.regs = fa.numRegs;
    vi.ready = true;
    return ALCS_OK;
}

int schedule_index_for_kc(const alcs_packed* w, int kc)
{
    for (int i = 0; i < alcs::kNumChunkings; ++i)
        if (w->sched[i].seg_ptr && w->sched[i].kc == kc) return i;
    return -1;
}

using alcs::Plan;

size_t plan_smem(const KernelVariant& v, int kc, int nch, int stages, int elt)
{
    return (size_t)std::min(stages, nch) * kc * 32 * v.p * elt;
}

// A rough per-layer time model (seconds) used to rank launch configurations.  Three resources
// are modelled per SM: FMA issue slots, shared-memory/L1 wavefronts and bytes from L2; plus the
// HBM floor and the quantisation of thread blocks into waves.
double model_cost(const alcs_packed* w, const KernelVariant& v, const alcs::DeviceSchedule& sc,
                  int stages, int n_rg, int rows_per_rg, long long q, int sms, int occ)
{
    const int elt = (int)w->elt();
    const int T = 32 * v.p;
    const long long n_tiles = (q + T - 1) / T;
    const long long ctas = n_tiles * n_rg;
    const long long slots = (long long)sms * occ;
    const long long waves = (ctas + slots - 1) / slots;
    const int vg = (v.p * elt >= 16) ? 16 / elt : v.p;
    const int ng = v.p / vg;
    const double blocks_cta = (double)sc.nbp * rows_per_rg / std::max(1, w->rows);
    const double seg_cta = (double)rows_per_rg * sc.nch;
    const double fma_issue = blocks_cta * (v.g * v.p + ng + 2.5 + (elt == 2 ? v.p / 2 : 0)) / 4.0 + seg_cta * 12.0 / 4.0;
    const double lsu = blocks_cta * (ng * (vg * elt * 32 / 128.0) + 1.5) + (double)sc.nch * sc.kc * T * elt / 128.0;
    const double l2_bytes_cta = (double)std::min(w->cin, sc.nch * sc.kc) * T * elt;
    const double l2 = l2_bytes_cta / 48.0;   // ~48 B/clk/SM sustained from L2
    // latency hiding: with few resident warps the pipes are not kept busy
    const double warps = (double)v.nw * occ;
    const double hide = std::min(1.0, 0.45 + warps / 28.0);
    const double cta_cycles = std::max(std::max(fma_issue, lsu), l2) / hide + 2500.0 / occ;
    const double clock = 1.9e9;
    const double t_sm = (double)waves * occ * cta_cycles / clock;
    const double bytes = (double)q * (w->cin + w->cout) * elt;
    const double t_hbm = bytes / 6.0e12;
    return std::max(t_sm, t_hbm);
}

int occupancy_of(const VariantInfo& vi, size_t smem)
{
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, vi.v.fn, vi.v.nw * 32, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return occ;
}

// Enumerate every valid launch configuration for this shape, cheapest (by the model) first.
int enumerate_plans(const alcs_packed* w, long long q, std::vector<Plan>& out)
{
    DeviceInfo di;
    int rc = device_info(w->device, &di);
    if (rc) return rc;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        init_variants_locked();
    }
    const int elt = (int)w->elt();
    out.clear();
    for (size_t vi = 0; vi < g_variants.size(); ++vi) {
        const KernelVariant& v = g_variants[vi].v;
        if (v.is_f16 != (w->dt == ALCS_F16) || v.g != w->g) continue;
        rc = prepare_variant(g_variants[vi]);
        if (rc) return rc;
        const int cap = v.nw * v.rw;
        const int rg_min = (w->rows + cap - 1) / cap;
        for (int si = 0; si < alcs::kNumChunkings; ++si) {
            const alcs::DeviceSchedule& sc = w->sched[si];
            if (!sc.seg_ptr) continue;
            for (int stages = 2; stages <= 4; ++stages) {
                if (stages > 2 && sc.nch < stages) continue;
                const size_t smem = plan_smem(v, sc.kc, sc.nch, stages, elt);
                if (smem > (size_t)std::min(kMaxSmem, di.smem_optin)) continue;
                const int occ = occupancy_of(g_variants[vi], smem);
                if (occ < 1) continue;
                int last_rpg = -1;
                for (int n_rg = rg_min; n_rg <= std::min(w->rows, rg_min * 4 + 2); ++n_rg) {
                    const int rpg = (w->rows + n_rg - 1) / n_rg;
                    if (rpg == last_rpg) continue;
                    last_rpg = rpg;
                    const int n_rg_eff = (w->rows + rpg - 1) / rpg;
                    Plan p;
                    p.variant = (int)vi; p.sched = si; p.stages = stages;
                    p.n_rg = n_rg_eff; p.rows_per_rg = rpg; p.smem = smem;
                    p.cost = model_cost(w, v, sc, stages, n_rg_eff, rpg, q, di.sms, occ);
                    out.push_back(p);
                }
            }
        }
    }
    std::stable_sort(out.begin(), out.end(), [](const Plan& a, const Plan& b) { return a.cost < b.cost; });
    return out.empty() ? ALCS_ERR_UNSUPPORTED : ALCS_OK;
}

void plan_to_cfg(const alcs_packed* w, const Plan& p, alcs_launch_cfg* c)
{
    const KernelVariant& v = g_variants[p.variant].v;
    c->pixels_per_lane = v.p;
    c->rows_per_warp = v.rw;
    c->warps = v.nw;
    c->chunk_channels = w->sched[p.sched].kc;
    c->stages = p.stages;
    c->row_groups = p.n_rg;
    c->min_blocks = v.minb;
}

// Resolve a (possibly partial) configuration into a concrete plan.
int cfg_to_plan(const alcs_packed* w, long long q, const alcs_launch_cfg* c, Plan* out)
{
    std::vector<Plan> all;
    int rc = enumerate_plans(w, q, all);
    if (rc) return rc;
    if (!c) { *out = all[0]; return ALCS_OK; }
    for (const Plan& p : all) {
        const KernelVariant& v = g_variants[p.variant].v;
        if (c->pixels_per_lane && c->pixels_per_lane != v.p) continue;
        if (c->rows_per_warp && c->rows_per_warp != v.rw) continue;
        if (c->warps && c->warps != v.nw) continue;
        if (c->min_blocks && c->min_blocks != v.minb) continue;
        if (c->chunk_channels && c->chunk_channels != w->sched[p.sched].kc) continue;
        if (c->stages && c->stages != p.stages) continue;
        if (c->row_groups && c->row_groups != p.n_rg) continue;
        *out = p;
        return ALCS_OK;
    }
    // row_groups outside the enumerated range: accept any feasible count for a matching variant
    if (c->row_groups > 0) {
        for (const Plan& p0 : all) {
            const KernelVariant& v = g_variants[p0.variant].v;
            if (c->pixels_per_lane && c->pixels_per_lane != v.p) continue;
            if (c->rows_per_warp && c->rows_per_warp != v.rw) continue;
            if (c->warps && c->warps != v.nw) continue;
            if (c->min_blocks && c->min_blocks != v.minb) continue;
            if (c->chunk_channels && c->chunk_channels != w->sched[p0.sched].kc) continue;
            if (c->stages && c->stages != p0.stages) continue;
            const int rpg = (w->rows + c->row_groups - 1) / c->row_groups;
            if (rpg > v.nw * v.rw) continue;
            Plan p = p0;
            p.rows_per_rg = rpg;
            p.n_rg = (w->rows + rpg - 1) / rpg;
            *out = p;
            return ALCS_OK;
        }
    }
    return ALCS_ERR_UNSUPPORTED;
}

int check_conv_args(const alcs_packed* w, const void* x, const void* y, int n, int h, int wd,
                    unsigned flags, long long* q_out)
{
    if (!w) return ALCS_ERR_INVALID_ARG;
    if (n < 0 || h < 0 || wd < 0) return ALCS_ERR_INVALID_ARG;
    if (flags & ~(ALCS_RELU | ALCS_Y_F32)) return ALCS_ERR_INVALID_ARG;
    if ((flags & ALCS_Y_F32) && w->dt != ALCS_F16) return ALCS_ERR_INVALID_ARG;
    if (w->g != 1 && w->g != 2 && w->g != 4 && w->g != 8 && w->g != 16) return ALCS_ERR_UNSUPPORTED;
    const long long hw = (long long)h * wd;
    const long long q = hw * n;
    if (hw > (1ll << 30) || q > (1ll << 30)) return ALCS_ERR_SHAPE;
    *q_out = q;
    if (q == 0) return ALCS_OK;
    if (!x || !y) return ALCS_ERR_INVALID_ARG;
    const size_t xe = w->elt(), ye = (w->dt == ALCS_F16 && !(flags & ALCS_Y_F32)) ? 2 : 4;
    if ((uintptr_t)x % xe || (uintptr_t)y % ye) return ALCS_ERR_INVALID_ARG;
    const uintptr_t xb = (uintptr_t)x, xend = xb + (size_t)q * w->cin * xe;
    const uintptr_t yb = (uintptr_t)y, yend = yb + (size_t)q * w->cout * ye;
    if (xb < yend && yb < xend) return ALCS_ERR_INVALID_ARG;   // x and y overlap
    return ALCS_OK;
}

int launch_plan(const alcs_packed* w, const Plan& p, const void* x, void* y, int n, int h, int wd,
                const float* bias, unsigned flags, cudaStream_t st)
{
    const KernelVariant& v = g_variants[p.variant].v;
    const alcs::DeviceSchedule& sc = w->sched[p.sched];
    const int elt = (int)w->elt();
    const int hw = h * wd;
    ConvArgs a;
    a.x = x; a.y = y; a.bias = bias;
    a.seg_ptr = sc.seg_ptr; a.cols = sc.cols; a.vals = sc.vals; a.row_order = w->d_row_order;
    a.rows = w->rows; a.cin = w->cin; a.cout = w->cout; a.hw = hw;
    a.q_total = n * hw;
    a.n_rg = p.n_rg; a.rows_per_rg = p.rows_per_rg;
    a.kc = sc.kc; a.nch = sc.nch; a.stages = p.stages;
    a.relu = (flags & ALCS_RELU) ? 1 : 0;
    a.y_f32 = (flags & ALCS_Y_F32) ? 1 : 0;
    // widest staging copy that every (image, channel) row start and length allows
    int ld = 16;
    while (ld > elt && (((size_t)hw * elt) % ld || (uintptr_t)x % ld)) ld >>= 1;
    a.ld_bytes = ld;
    const int vg = (v.p * elt >= 16) ? 16 / elt : v.p;
    a.st_vec = (hw % vg == 0 && (uintptr_t)y % 16 == 0) ? 1 : 0;
    const int T = 32 * v.p;
    const long long n_tiles = ((long long)a.q_total + T - 1) / T;
    const long long grid = n_tiles * p.n_rg;
    if (grid > 0x7fffffffll) return ALCS_ERR_SHAPE;
    void* args[] = {&a};
    ALCS_CUDA(cudaLaunchKernel(v.fn, dim3((unsigned)grid), dim3(v.nw * 32), args, p.smem, st));
    return ALCS_OK;
}

int check_device(const alcs_packed* w)
{
    if (w->device < 0) return ALCS_ERR_STATE;
    int cur = -1;
    ALCS_CUDA(cudaGetDevice(&cur));
    return cur == w->device ? ALCS_OK : ALCS_ERR_STATE;
}

int resolve_plan(const alcs_packed* w, int n, int h, int wd, unsigned flags, long long q,
                 const alcs_launch_cfg* cfg, Plan* plan)
{
    if (cfg) return cfg_to_plan(w, q, cfg, plan);
    const alcs::ShapeKey key{n, h, wd, flags};
    {
        std::lock_guard<std::mutex> lk(w->mu);
        auto it = w->plan_cache.find(key);
        if (it != w->plan_cache.end()) { *plan = it->second; return ALCS_OK; }
    }
    auto it = w->tuned.find(key);
    const int rc = cfg_to_plan(w, q, it != w->tuned.end() ? &it->second : nullptr, plan);
    if (rc) return rc;
    std::lock_guard<std::mutex> lk(w->mu);
    w->plan_cache[key] = *plan;
    return ALCS_OK;
}

}  // namespace

struct alcs_stack {
    struct Item {
        alcs_layer layer;
        Plan plan;
        long long q;
    };
    std::vector<Item> items;
    unsigned flags = 0;
    cudaGraphExec_t exec = nullptr;
};

extern "C" {

ALCS_API int alcs_packed_upload(alcs_packed* p, int device, void* cuda_stream)
{
    if (!p) return ALCS_ERR_INVALID_ARG;
    if (p->device >= 0) return ALCS_ERR_STATE;
    int ndev = 0;
    ALCS_CUDA(cudaGetDeviceCount(&ndev));
    if (device < 0 || device >= ndev) return ALCS_ERR_INVALID_ARG;
    int prev = -1;
    ALCS_CUDA(cudaGetDevice(&prev));
    ALCS_CUDA(cudaSetDevice(device));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int rc = ALCS_OK;
    std::vector<alcs::HostSchedule> hs(alcs::kNumChunkings);
    std::vector<int> order;
    auto fail = [&](int code) {
        for (auto& s : p->sched) {
            cudaFree(s.seg_ptr); cudaFree(s.cols); cudaFree(s.vals);
            s = alcs::DeviceSchedule();
        }
        cudaFree(p->d_row_order);
        p->d_row_order = nullptr;
        (void)cudaGetLastError();
        cudaSetDevice(prev);
        return code;
    };
    try {
        alcs::build_row_order(*p, order);
        for (int i = 0; i < alcs::kNumChunkings; ++i) {
            int kc = alcs::kChunkings[i];
            if (kc == 0 || kc > p->cin) kc = p->cin;
            bool dup = false;
            for (int j = 0; j < i; ++j) dup |= (hs[j].kc == kc);
            if (dup) { hs[i].kc = -1; continue; }
            alcs::build_schedule(*p, kc, hs[i]);
        }
    } catch (const std::bad_alloc&) {
        return fail(ALCS_ERR_ALLOC);
    }
#define UP_CUDA(call)                                              \
    do {                                                           \
        cudaError_t e_ = (call);                                   \
        if (e_ != cudaSuccess) {                                   \
            alcs::set_cuda_error_text(cudaGetErrorString(e_));     \
            return fail(e_ == cudaErrorMemoryAllocation ? ALCS_ERR_ALLOC : ALCS_ERR_CUDA); \
        }                                                          \
    } while (0)
    UP_CUDA(cudaMalloc(&p->d_row_order, std::max<size_t>(4, order.size() * 4)));
    UP_CUDA(cudaMemcpyAsync(p->d_row_order, order.data(), order.size() * 4, cudaMemcpyHostToDevice, st));
    for (int i = 0; i < alcs::kNumChunkings; ++i) {
        if (hs[i].kc < 0) continue;
        alcs::DeviceSchedule& d = p->sched[i];
        d.kc = hs[i].kc; d.nch = hs[i].nch; d.nbp = hs[i].nbp;
        UP_CUDA(cudaMalloc(&d.seg_ptr, hs[i].seg_ptr.size() * 4));
        UP_CUDA(cudaMalloc(&d.cols, std::max<size_t>(16, hs[i].cols.size() * 4)));
        UP_CUDA(cudaMalloc(&d.vals, std::max<size_t>(16, hs[i].vals.size() * 4)));
        UP_CUDA(cudaMemcpyAsync(d.seg_ptr, hs[i].seg_ptr.data(), hs[i].seg_ptr.size() * 4, cudaMemcpyHostToDevice, st));
        if (!hs[i].cols.empty()) {
            UP_CUDA(cudaMemcpyAsync(d.cols, hs[i].cols.data(), hs[i].cols.size() * 4, cudaMemcpyHostToDevice, st));
            UP_CUDA(cudaMemcpyAsync(d.vals, hs[i].vals.data(), hs[i].vals.size() * 4, cudaMemcpyHostToDevice, st));
        }
    }
    UP_CUDA(cudaStreamSynchronize(st));
#undef UP_CUDA
    p->device = device;
    cudaSetDevice(prev);
    return rc;
}

ALCS_API void alcs_packed_free(alcs_packed* p)
{
    if (!p) return;
    if (p->device >= 0) {
        int prev = -1;
        if (cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(p->device) == cudaSuccess) {
            for (auto& s : p->sched) { cudaFree(s.seg_ptr); cudaFree(s.cols); cudaFree(s.vals); }
            cudaFree(p->d_row_order);
            cudaSetDevice(prev);
        }
        (void)cudaGetLastError();
    }
    delete p;
}

ALCS_API int alcs_variant_count(void)
{
    std::lock_guard<std::mutex> lk(g_mu);
    init_variants_locked();
    return (int)g_variants.size();
}

ALCS_API int alcs_variant_get(int index, alcs_dtype* dt, int* g, alcs_launch_cfg* cfg)
{
    std::lock_guard<std::mutex> lk(g_mu);
    init_variants_locked();
    if (index < 0 || index >= (int)g_variants.size()) return ALCS_ERR_INVALID_ARG;
    const KernelVariant& v = g_variants[index].v;
    if (dt) *dt = v.is_f16 ? ALCS_F16 : ALCS_F32;
    if (g) *g = v.g;
    if (cfg) {
        std::memset(cfg, 0, sizeof *cfg);
        cfg->pixels_per_lane = v.p;
        cfg->rows_per_warp = v.rw;
        cfg->warps = v.nw;
        cfg->min_blocks = v.minb;
    }
    return ALCS_OK;
}

ALCS_API int alcs_spconv1x1_cfg(const alcs_packed* w, const void* x, void* y, int n, int h, int wd,
                       const float* bias, unsigned flags, const alcs_launch_cfg* cfg,
                       void* cuda_stream)
{
    long long q = 0;
    int rc = check_conv_args(w, x, y, n, h, wd, flags, &q);
    if (rc) return rc;
    rc = check_device(w);
    if (rc) return rc;
    if (q == 0) return ALCS_OK;
    Plan plan;
    rc = resolve_plan(w, n, h, wd, flags, q, cfg, &plan);
    if (rc) return rc;
    return launch_plan(w, plan, x, y, n, h, wd, bias, flags, static_cast<cudaStream_t>(cuda_stream));
}

ALCS_API int alcs_spconv1x1(const alcs_packed* w, const void* x, void* y, int n, int h, int wd,
                   const float* bias, unsigned flags, void* cuda_stream)
{
    return alcs_spconv1x1_cfg(w, x, y, n, h, wd, bias, flags, nullptr, cuda_stream);
}

ALCS_API int alcs_spconv1x1_plan(const alcs_packed* w, int n, int h, int wd, unsigned flags,
                        alcs_launch_cfg* out)
{
    if (!w || !out || n < 0 || h < 0 || wd < 0) return ALCS_ERR_INVALID_ARG;
    if (flags & ~(ALCS_RELU | ALCS_Y_F32)) return ALCS_ERR_INVALID_ARG;
    if ((flags & ALCS_Y_F32) && w->dt != ALCS_F16) return ALCS_ERR_INVALID_ARG;
    if (w->g != 1 && w->g != 2 && w->g != 4 && w->g != 8 && w->g != 16) return ALCS_ERR_UNSUPPORTED;
    if (w->device < 0) return ALCS_ERR_STATE;
    const long long q = (long long)n * h * wd;
    if ((long long)h * wd > (1ll << 30) || q > (1ll << 30)) return ALCS_ERR_SHAPE;
    Plan plan;
    const int rc = resolve_plan(w, n, h, wd, flags, std::max(1ll, q), nullptr, &plan);
    if (rc) return rc;
    plan_to_cfg(w, plan, out);
    return ALCS_OK;
}

ALCS_API int alcs_spconv1x1_tune(alcs_packed* w, const void* x, void* y, int n, int h, int wd,
                        const float* bias, unsigned flags, void* cuda_stream,
                        alcs_launch_cfg* best)
{
    long long q = 0;
    int rc = check_conv_args(w, x, y, n, h, wd, flags, &q);
    if (rc) return rc;
    rc = check_device(w);
    if (rc) return rc;
    if (q == 0) return ALCS_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    std::vector<Plan> all;
    rc = enumerate_plans(w, q, all);
    if (rc) return rc;
    const size_t max_try = 48;
    if (all.size() > max_try) all.resize(max_try);
    // a buffer larger than L2, rewritten before every timed launch so that each candidate is
    // timed with cold caches, as it will run inside a network
    const size_t flush_bytes = 256u << 20;
    void* flush = nullptr;
    if (cudaMalloc(&flush, flush_bytes) != cudaSuccess) { (void)cudaGetLastError(); flush = nullptr; }
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    auto cleanup = [&]() {
        if (e0) cudaEventDestroy(e0);
        if (e1) cudaEventDestroy(e1);
        if (flush) cudaFree(flush);
    };
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        cleanup();
        alcs::set_cuda_error_text("cudaEventCreate failed");
        return ALCS_ERR_CUDA;
    }
    int best_i = -1;
    float best_ms = 1e30f;
    const int reps = 3;
    for (size_t i = 0; i < all.size(); ++i) {
        float tmin = 1e30f;
        bool ok = true;
        for (int r = 0; r < reps + 1 && ok; ++r) {
            if (flush) cudaMemsetAsync(flush, r, flush_bytes, st);
            cudaEventRecord(e0, st);
            ok = launch_plan(w, all[i], x, y, n, h, wd, bias, flags, st) == ALCS_OK;
            cudaEventRecord(e1, st);
            if (cudaEventSynchronize(e1) != cudaSuccess) { ok = false; break; }
            float ms = 0;
            cudaEventElapsedTime(&ms, e0, e1);
            if (r > 0) tmin = std::min(tmin, ms);
        }
        if (ok && tmin < best_ms) { best_ms = tmin; best_i = (int)i; }
    }
    cudaError_t e = cudaStreamSynchronize(st);
    cleanup();
    if (e != cudaSuccess) { alcs::set_cuda_error_text(cudaGetErrorString(e)); return ALCS_ERR_CUDA; }
    if (best_i < 0) return ALCS_ERR_CUDA;
    alcs_launch_cfg c;
    plan_to_cfg(w, all[best_i], &c);
    {
        std::lock_guard<std::mutex> lk(w->mu);
        w->tuned[alcs::ShapeKey{n, h, wd, flags}] = c;
        w->plan_cache[alcs::ShapeKey{n, h, wd, flags}] = all[best_i];
    }
    // leave y holding the result of the chosen configuration
    rc = launch_plan(w, all[best_i], x, y, n, h, wd, bias, flags, st);
    if (best) *best = c;
    return rc;
}

ALCS_API size_t alcs_spconv1x1_host_workspace(const alcs_packed* w, int n, int h, int wd, unsigned flags)
{
    if (!w || n < 0 || h < 0 || wd < 0) return 0;
    const size_t q = (size_t)n * h * wd;
    const size_t ye = (w->dt == ALCS_F16 && !(flags & ALCS_Y_F32)) ? 2 : 4;
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    return up(q * w->cin * w->elt()) + up(q * w->cout * ye) + up((size_t)w->cout * 4);
}

ALCS_API int alcs_spconv1x1_host(const alcs_packed* w, const void* x_host, void* y_host, int n, int h,
                        int wd, const float* bias_host, unsigned flags, void* workspace,
                        size_t workspace_bytes, void* cuda_stream)
{
    if (!w || !workspace || (uintptr_t)workspace % 256) return ALCS_ERR_INVALID_ARG;
    if (n < 0 || h < 0 || wd < 0) return ALCS_ERR_INVALID_ARG;
    const size_t need = alcs_spconv1x1_host_workspace(w, n, h, wd, flags);
    if (workspace_bytes < need) return ALCS_ERR_SHAPE;
    const size_t q = (size_t)n * h * wd;
    if (q == 0) return ALCS_OK;
    if (!x_host || !y_host) return ALCS_ERR_INVALID_ARG;
    const size_t ye = (w->dt == ALCS_F16 && !(flags & ALCS_Y_F32)) ? 2 : 4;
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t xb = q * w->cin * w->elt(), yb = q * w->cout * ye;
    unsigned char* dx = static_cast<unsigned char*>(workspace);
    unsigned char* dy = dx + up(xb);
    float* db = reinterpret_cast<float*>(dy + up(yb));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int rc = check_device(w);
    if (rc) return rc;
    ALCS_CUDA(cudaMemcpyAsync(dx, x_host, xb, cudaMemcpyHostToDevice, st));
    if (bias_host) ALCS_CUDA(cudaMemcpyAsync(db, bias_host, (size_t)w->cout * 4, cudaMemcpyHostToDevice, st));
    rc = alcs_spconv1x1(w, dx, dy, n, h, wd, bias_host ? db : nullptr, flags, cuda_stream);
    if (rc) return rc;
    ALCS_CUDA(cudaMemcpyAsync(y_host, dy, yb, cudaMemcpyDeviceToHost, st));
    return ALCS_OK;
}

ALCS_API int alcs_stack_create(const alcs_layer* layers, int n_layers, unsigned stack_flags, alcs_stack** out)
{
    if (!out) return ALCS_ERR_INVALID_ARG;
    *out = nullptr;
    if (!layers || n_layers < 0 || (stack_flags & ~ALCS_STACK_GRAPH)) return ALCS_ERR_INVALID_ARG;
    alcs_stack* s = new (std::nothrow) alcs_stack();
    if (!s) return ALCS_ERR_ALLOC;
    s->flags = stack_flags;
    for (int i = 0; i < n_layers; ++i) {
        const alcs_layer& L = layers[i];
        alcs_stack::Item it;
        it.layer = L;
        int rc = check_conv_args(L.w, L.x, L.y, L.n, L.h, L.wd, L.flags, &it.q);
        if (!rc) rc = check_device(L.w);
        if (!rc && it.q > 0) rc = resolve_plan(L.w, L.n, L.h, L.wd, L.flags, it.q, nullptr, &it.plan);
        if (rc) { delete s; return rc; }
        s->items.push_back(it);
    }
    *out = s;
    return ALCS_OK;
}

static int stack_enqueue(alcs_stack* s, cudaStream_t st)
{
    for (auto& it : s->items) {
        if (it.q == 0) continue;
        const alcs_layer& L = it.layer;
        int rc = launch_plan(L.w, it.plan, L.x, L.y, L.n, L.h, L.wd, L.bias, L.flags, st);
        if (rc) return rc;
    }
    return ALCS_OK;
}

ALCS_API int alcs_stack_run(alcs_stack* s, void* cuda_stream)
{
    if (!s) return ALCS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (!(s->flags & ALCS_STACK_GRAPH)) return stack_enqueue(s, st);
    if (!s->exec) {
        cudaStream_t cap = nullptr;
        // capture on a private stream so that the caller's stream may be the legacy default one
        ALCS_CUDA(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking));
        cudaGraph_t graph = nullptr;
        cudaError_t e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
        int rc = ALCS_OK;
        if (e == cudaSuccess) {
            rc = stack_enqueue(s, cap);
            e = cudaStreamEndCapture(cap, &graph);
        }
        if (e == cudaSuccess && rc == ALCS_OK) e = cudaGraphInstantiate(&s->exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
        cudaStreamDestroy(cap);
        if (rc) return rc;
        if (e != cudaSuccess) {
            alcs::set_cuda_error_text(cudaGetErrorString(e));
            (void)cudaGetLastError();
            s->exec = nullptr;
            return ALCS_ERR_CUDA;
        }
    }
    ALCS_CUDA(cudaGraphLaunch(s->exec, st));
    return ALCS_OK;
}

ALCS_API int alcs_stack_destroy(alcs_stack* s)
{
    if (!s) return ALCS_OK;
    if (s->exec) cudaGraphExecDestroy(s->exec);
    delete s;
    return ALCS_OK;
}

}  // extern "C"
