// Compiled variants of the general k x k sparse convolution kernel (fp32) and their launcher.
#include "alcs_conv2d.cuh"

#include <algorithm>
#include <array>
#include <cstring>
#include <mutex>
#include <new>

#include "alcs_internal.h"

namespace alcs {
void set_cuda_error_text(const char* s);
}

namespace alcs {

namespace {

struct Conv2dVariant {
    int g, p, st, ni;
    const void* fn[2];      // [0] all channels in one chunk, [1] chunked
    bool ready[2][64];      // by device: the shared-memory attribute is set per device
};

#define ALCS_C2D_N(G, P, ST, NI)                                                            \
    {G, P, ST, NI, {(const void*)&spconv2d_kernel<G, P, ST, kConv2dWarps, false, NI>,       \
                    (const void*)&spconv2d_kernel<G, P, ST, kConv2dWarps, true, NI>}, {}}
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
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lk(g_c2d_mu);
        if (!v->ready[ch][dev]) {
            e = cudaFuncSetAttribute(v->fn[ch], cudaFuncAttributeMaxDynamicSharedMemorySize, kConv2dMaxDynSmem);
            if (e != cudaSuccess) return e;
            v->ready[ch][dev] = true;
        }
    }
    Conv2dArgs args = a;
    void* params[] = {&args};
    return cudaLaunchKernel(v->fn[ch], dim3(grid), dim3(kConv2dWarps * 32), params, smem, st);
}

}  // namespace alcs

// ---------------------------------------------------------------------------------------------
// General k x k convolution (paper, Section 3.2.2: the convolution formula with all three sums,
// seen as W* x I* with the columns of W* indexed by (c, r, s)).  Same packed format; the packed
// matrix has cin*kh*kw columns.
// ---------------------------------------------------------------------------------------------
namespace {

using alcs::Schedule;

#define ALCS_CUDA(call)                                        \
    do {                                                       \
        cudaError_t e_ = (call);                               \
        if (e_ != cudaSuccess) {                               \
            alcs::set_cuda_error_text(cudaGetErrorString(e_)); \
            (void)cudaGetLastError();                          \
            return ALCS_ERR_CUDA;                              \
        }                                                      \
    } while (0)

struct Conv2dGeom {
    int n, cin, h, wd, kh, kw, st, pad, oh, ow;
};

struct Conv2dPlan {
    int p = 0;          // positions per lane
    int th = 0;         // output rows per strip
    int n_strips = 0, n_rg = 0;
    int npt = 0, nrs = 0;
    int wp = 0, pr = 0, pl = 0, chw = 0, slack = 0;
    int kc = 0, nch = 0;     // input channels per chunk, chunks
    int ni = 1;              // images per work item
    size_t smem = 0;
    double cost = 0;    // model estimate, cycles per SM
};

// Choose positions per lane, strip height and row-group count by a small cost model: per work item
// the patch is staged once (element-wise copies, about 2 words per cycle per SM) and every kept block costs
// G*P*32 FMAs per position tile at the rate the shared-memory-bound hot loop sustains; items are
// dealt to one persistent thread block per SM.
int plan_conv2d(const alcs_packed* w, const Conv2dGeom& g, int sms, int smem_max, Conv2dPlan* out,
                const alcs_conv2d_cfg* force = nullptr)
{
    const int NW = alcs::kConv2dWarps;
    const int wp = g.ow + (g.kw - 1) / g.st;
    const int halo = (g.kh - 1) / g.st;
    Conv2dPlan best;
    best.cost = 1e300;
    for (int ni = 1; ni <= 4; ni *= 2)
    for (int p = 8; p >= 2; p /= 2) {
        if (!alcs::conv2d_variant_exists(w->g, p, g.st, ni)) continue;
        if (force && force->images_per_item && force->images_per_item != ni) continue;
        if (force && force->positions_per_lane && force->positions_per_lane != p) continue;
        // sustained fraction of the fp32 peak in the hot loop: per pair of blocks 2P X wavefronts
        // plus 3 of records against 16P/8 cycles of FMA issue
        const double rate = 128.0 * 0.6 * (2.0 * p / (2.0 * p + 3.0)) / (16.0 / 19.0);
        for (int th = 1; th <= g.oh; ++th) {
            if (force && force->strip_rows && force->strip_rows != th) continue;
            const int positions = th * wp;
            // several images per item: whole images only, each within its 32 * p / ni position slots
            if (ni > 1 && (th != g.oh || positions > 32 * p / ni)) continue;
            const int npt = ni > 1 ? 1 : (positions + 32 * p - 1) / (32 * p);
            if (npt > NW) break;
            const int pr = th + halo;
            const long long chw = (long long)g.st * g.st * pr * wp;
            const int slack = (ni > 1 ? 32 * p / ni : npt * 32 * p) - positions + 8;
            const int nrs = NW / npt;
            const int n_strips = (g.oh + th - 1) / th;
            const long long base_items = (long long)((g.n + ni - 1) / ni) * n_strips;
            // channels per chunk: all of them if the patch fits, else halves, quarters, ...
            for (int nch = 1; nch <= g.cin; nch *= 2) {
                const int kc = (force && force->chunk_channels) ? std::min(force->chunk_channels, g.cin) : (g.cin + nch - 1) / nch;
                const int nch_real = (g.cin + kc - 1) / kc;
                const long long smem = (((long long)kc * chw * ni + slack) * 4 + 15) / 16 * 16 + (long long)NW * alcs::rec_buffer_bytes(w->g);
                if (smem > smem_max) { if (force && force->chunk_channels) break; continue; }
                // one chunk: warps take rows from a counter, any number of row groups; several chunks:
                // one row per warp, so the row groups are fixed by the warps per position tile
                const int rg_fixed = (w->rows + nrs - 1) / nrs;
                const int rg_lo = nch_real == 1 ? 1 : rg_fixed;
                const int rg_hi = nch_real == 1 ? std::max(1, std::min(w->rows, 32)) : rg_fixed;
                for (int n_rg = rg_lo; n_rg <= rg_hi; ++n_rg) {
                    if (force && force->row_groups && nch_real == 1 && force->row_groups != n_rg) continue;
                    const long long items = base_items * n_rg;
                    const long long rounds = (items + sms - 1) / sms;
                    // (measured: the 4-byte staging copies sustain about 2 words per cycle and SM)
                    const double stage = (double)g.cin * chw * ni / 2.0 + 1500.0 * nch_real;
                    const double blocks_item = (double)w->nb / n_rg;
                    const double fma = blocks_item * npt * (double)(w->g * p * 32);
                    // warps that share a position tile split its rows; idle warps (NW not a multiple of
                    // npt) and a short row list (fewer rows than warps) leave lanes unused
                    const int rpg = (w->rows + n_rg - 1) / n_rg;
                    const double use = (double)(npt * std::min(nrs, rpg)) / NW;
                    const double compute = fma / (rate * use);
                    const double cost = rounds * (stage + compute + 3000.0);
                    if (cost < best.cost) {
                        best.p = p; best.th = th; best.n_strips = n_strips; best.n_rg = n_rg;
                        best.npt = npt; best.nrs = nrs; best.wp = wp; best.pr = pr; best.pl = pr * wp;
                        best.chw = (int)chw; best.slack = slack; best.smem = (size_t)smem; best.cost = cost;
                        best.kc = kc; best.nch = nch_real; best.ni = ni;
                    }
                }
                break;      // the largest chunk that fits is the one to use for this (p, th)
            }
        }
    }
    if (best.p == 0) return ALCS_ERR_UNSUPPORTED;     // not even a one-row strip of all channels fits
    *out = best;
    return ALCS_OK;
}

// The whole-row schedule (one chunk = all columns) with every column index replaced by the byte
// offset of that column's (channel, tap) inside the shared-memory patch.
Schedule* get_schedule2d(const alcs_packed* w, const Conv2dGeom& g, const Conv2dPlan& p)
{
    const int chs = p.chw * p.ni;      // words per channel of the staged patch
    const std::array<int, 8> key = {p.n_rg, chs, p.pl, p.wp, g.st, g.kh, g.kw, p.kc};
    std::lock_guard<std::mutex> lk(w->mu);
    auto it = w->sched2d.find(key);
    if (it != w->sched2d.end()) return &it->second;
    try {
        Schedule& sc = w->sched2d[key];
        const int taps = g.kh * g.kw;
        alcs::build_schedule(*w, p.kc * taps, p.n_rg, true, sc);      // chunk = kc channels = kc*taps columns
        auto coloff = [&](int col) {
            const int c = col / taps, tap = col - c * taps;
            const int r = tap / g.kw, s = tap - r * g.kw;
            return 4 * (c * chs + ((r % g.st) * g.st + (s % g.st)) * p.pl + (r / g.st) * p.wp + s / g.st);
        };
        const int REC = alcs::record_bytes(w->g);
        // (columns inside a chunk are chunk-local, and a chunk starts at a channel boundary, so the
        //  same formula gives the offset inside the staged chunk)
        for (int rgk = 0; rgk < sc.n_rg * sc.nch; ++rgk)
            for (int t = 0; t < sc.rpg; ++t) {
                int* hd = &sc.h_rowoff[(size_t)rgk * sc.ros + 4 * t];
                const int npairs = hd[3];
                if (npairs == 0) continue;
                hd[1] = coloff(hd[1]);
                hd[2] = coloff(hd[2]);
                unsigned char* base = &sc.h_rec[((size_t)sc.h_slice[rgk] + hd[0]) * 16];
                for (int q = 0; q < npairs; ++q) {
                    int hdr[2];
                    std::memcpy(hdr, base + (size_t)q * REC, 8);
                    hdr[0] = coloff(hdr[0]);
                    hdr[1] = coloff(hdr[1]);
                    std::memcpy(base + (size_t)q * REC, hdr, 8);
                }
            }
        return &sc;
    } catch (const std::bad_alloc&) {
        w->sched2d.erase(key);
        return nullptr;
    }
}

int check_conv2d_args(const alcs_packed* w, const void* x, const void* y, int n, int cin, int h, int wd, int kh,
                      int kw, int stride, int pad, unsigned flags, Conv2dGeom* g, bool with_buffers = true)
{
    if (!w) return ALCS_ERR_INVALID_ARG;
    if (n < 0 || cin <= 0 || h <= 0 || wd <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0) return ALCS_ERR_INVALID_ARG;
    if (flags & ~ALCS_RELU) return ALCS_ERR_INVALID_ARG;
    if ((long long)cin * kh * kw != w->cin) return ALCS_ERR_SHAPE;
    if (h + 2 * pad < kh || wd + 2 * pad < kw) return ALCS_ERR_SHAPE;
    if (w->dt != ALCS_F32) return ALCS_ERR_UNSUPPORTED;
    if (w->g != 1 && w->g != 2 && w->g != 4 && w->g != 8 && w->g != 16) return ALCS_ERR_UNSUPPORTED;
    if (stride > 2 || (kw - 1) / stride > 8) return ALCS_ERR_UNSUPPORTED;
    g->n = n; g->cin = cin; g->h = h; g->wd = wd; g->kh = kh; g->kw = kw; g->st = stride; g->pad = pad;
    g->oh = (h + 2 * pad - kh) / stride + 1;
    g->ow = (wd + 2 * pad - kw) / stride + 1;
    const long long xin = (long long)n * cin * h * wd, yout = (long long)n * w->cout * g->oh * g->ow;
    if (xin > (1ll << 31) - 1 || yout > (1ll << 31) - 1) return ALCS_ERR_SHAPE;
    if (n == 0 || !with_buffers) return ALCS_OK;
    if (!x || !y) return ALCS_ERR_INVALID_ARG;
    if ((uintptr_t)x % 4 || (uintptr_t)y % 4) return ALCS_ERR_INVALID_ARG;
    const uintptr_t xb = (uintptr_t)x, xend = xb + (size_t)xin * 4, yb = (uintptr_t)y, yend = yb + (size_t)yout * 4;
    if (xb < yend && yb < xend) return ALCS_ERR_INVALID_ARG;
    return ALCS_OK;
}

}  // namespace

extern "C" ALCS_API int alcs_spconv2d_plan(const alcs_packed* w, int n, int cin, int h, int wd, int kh, int kw,
                                           int stride, int pad, alcs_conv2d_cfg* out)
{
    if (!out) return ALCS_ERR_INVALID_ARG;
    Conv2dGeom g;
    int rc = check_conv2d_args(w, nullptr, nullptr, n, cin, h, wd, kh, kw, stride, pad, 0, &g, false);
    if (rc) return rc;
    if (w->device < 0) return ALCS_ERR_STATE;
    int sms = 0, smem_optin = 0;
    rc = alcs::device_limits(w->device, &sms, &smem_optin);
    if (rc) return rc;
    Conv2dPlan p;
    rc = plan_conv2d(w, g, sms, std::min(alcs::kConv2dMaxDynSmem, smem_optin - 256), &p);
    if (rc) return rc;
    out->positions_per_lane = p.p; out->strip_rows = p.th; out->row_groups = p.n_rg;
    out->position_tiles = p.npt; out->warps_per_tile = p.nrs; out->smem_bytes = (int)p.smem;
    out->chunk_channels = p.kc; out->images_per_item = p.ni;
    return ALCS_OK;
}

extern "C" ALCS_API int alcs_spconv2d_cfg(const alcs_packed* w, const void* x, void* y, int n, int cin, int h, int wd,
                                          int kh, int kw, int stride, int pad, const float* bias, unsigned flags,
                                          const alcs_conv2d_cfg* cfg, void* cuda_stream)
{
    Conv2dGeom g;
    int rc = check_conv2d_args(w, x, y, n, cin, h, wd, kh, kw, stride, pad, flags, &g);
    if (rc) return rc;
    rc = alcs::require_current_device(w);
    if (rc) return rc;
    if (n == 0) return ALCS_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int sms = 0, smem_optin = 0;
    rc = alcs::device_limits(w->device, &sms, &smem_optin);
    if (rc) return rc;
    Conv2dPlan p;
    rc = plan_conv2d(w, g, sms, std::min(alcs::kConv2dMaxDynSmem, smem_optin - 256), &p, cfg);
    if (rc) return rc;
    Schedule* sc = get_schedule2d(w, g, p);
    if (!sc) return ALCS_ERR_ALLOC;
    if (!sc->uploaded) {
        rc = alcs::schedule_upload(w, sc, st);
        if (rc) return rc;
    }
    alcs::Conv2dArgs a;
    a.x = static_cast<const float*>(x); a.y = static_cast<float*>(y); a.bias = bias;
    a.rec = sc->rec; a.slice = sc->slice; a.rowoff = sc->rowoff; a.rowmap = sc->rowmap;
    a.rows = w->rows; a.cin = cin; a.cout = w->cout;
    a.h = h; a.wd = wd; a.oh = g.oh; a.ow = g.ow; a.kh = kh; a.kw = kw; a.pad = pad;
    a.th = p.th; a.n_strips = p.n_strips; a.n_rg = sc->n_rg; a.rpg = sc->rpg; a.n_img = n;
    a.wp = p.wp; a.pr = p.pr; a.pl = p.pl; a.chw = p.chw; a.npt = p.npt; a.nrs = p.nrs; a.slack = p.slack;
    a.kc = p.kc; a.nch = sc->nch;
    a.chs = p.chw * p.ni; a.n_igrp = (n + p.ni - 1) / p.ni;
    a.off_wbuf = (int)(((size_t)p.kc * a.chs + p.slack) * 4 + 15) / 16 * 16;
    if (sc->nch != p.nch || (sc->nch > 1 && sc->rpg > p.nrs)) return ALCS_ERR_STATE;      // (cannot happen: plan and schedule agree)
    a.relu = (flags & ALCS_RELU) ? 1 : 0;
    const long long items = (long long)a.n_igrp * p.n_strips * sc->n_rg;
    if (items > 0x7fffffffll) return ALCS_ERR_SHAPE;
    const unsigned grid = (unsigned)std::min<long long>(items, sms);
    ALCS_CUDA(alcs::launch_conv2d(w->g, p.p, stride, p.ni, a, grid, p.smem, st));
    return ALCS_OK;
}

extern "C" ALCS_API int alcs_spconv2d(const alcs_packed* w, const void* x, void* y, int n, int cin, int h, int wd,
                                      int kh, int kw, int stride, int pad, const float* bias, unsigned flags,
                                      void* cuda_stream)
{
    return alcs_spconv2d_cfg(w, x, y, n, cin, h, wd, kh, kw, stride, pad, bias, flags, nullptr, cuda_stream);
}
