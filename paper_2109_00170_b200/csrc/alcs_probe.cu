// Measurement probes of libalcs: small kernels that time, on the device they run on, the resources
// the pointwise kernel's hot loop (paper, Section 3.2.2, "Efficient multiplication computation")
// depends on.  They answer three questions with numbers instead of data-sheet arithmetic:
//   alcs_probe_fma_peak      what fp32 FMA rate do the CUDA cores reach from registers (the
//                            denominator of the ALU roofline);
//   alcs_probe_lds           what does a shared-memory load cost the SM's load/store pipe, for loads
//                            where every lane has its own address and for warp-uniform (broadcast) ones;
//   alcs_probe_segment_loop  what fraction of the fp32 peak does the kernel's own segment loop
//                            (consume_segment, compiled exactly as in the kernel) reach when all its
//                            data already sits in shared memory and nothing else runs.
// Each probe launches one thread block per SM, times the launch with CUDA events on the given
// stream (best of three after a warm-up) and synchronises that stream.
#include <cuda_runtime.h>

#include <cstring>
#include <vector>

#include "alcs_internal.h"
#include "alcs_kernels.cuh"

namespace alcs {
void set_cuda_error_text(const char* s);
}

namespace {

#define PROBE_CUDA(call)                                       \
    do {                                                       \
        cudaError_t e_ = (call);                               \
        if (e_ != cudaSuccess) {                               \
            alcs::set_cuda_error_text(cudaGetErrorString(e_)); \
            (void)cudaGetLastError();                          \
            return ALCS_ERR_CUDA;                              \
        }                                                      \
    } while (0)

// 32 independent dependent chains per thread, operands in registers.
__global__ void __launch_bounds__(512, 1) probe_ffma_kernel(float* out, int iters, float a, float b)
{
    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = threadIdx.x + i;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[i] = fmaf(acc[i], a, b);
    }
    float s = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) s += acc[i];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

__global__ void __launch_bounds__(512, 1) probe_ffma2_kernel(float* out, int iters, float a, float b)
{
    float2 acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = make_float2(threadIdx.x + i, i);
    const float2 a2 = make_float2(a, a), b2 = make_float2(b, b);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[i] = __ffma2_rn(acc[i], a2, b2);
    }
    float s = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) s += acc[i].x + acc[i].y;
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// Shared-memory loads only (one add per load keeps them alive): W bytes per lane, every lane its own
// address (conflict-free) or all lanes the same address.
template <int W, bool UNI>
__global__ void __launch_bounds__(512, 1) probe_lds_kernel(float* out, int iters)
{
    extern __shared__ __align__(16) unsigned char sm[];
    for (int i = threadIdx.x; i < 16384; i += blockDim.x) reinterpret_cast<float*>(sm)[i] = i;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const unsigned base = (unsigned)__cvta_generic_to_shared(sm) + (UNI ? 0 : lane * W) + (threadIdx.x >> 5) * 2048;
    float s = 0;
    unsigned off = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            const unsigned ad = base + ((off + u * 32 * W) & 0x3ff0);
            if constexpr (W == 16) {
                float4 v;
                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(ad));
                s += v.x;
            } else if constexpr (W == 8) {
                float2 v;
                asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(ad));
                s += v.x;
            } else {
                float v;
                asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(ad));
                s += v;
            }
        }
        off += 16;
    }
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace

namespace {

// The kernel's segment loop on synthetic segments that are resident in shared memory:
// [X tile of 64 channels x 32*P pixels | nseg segments of L pair records | nseg row headers].
// Every warp walks the segments in turn (RW accumulator sets, as the kernel's consumer warps do);
// columns are pseudo-random, so the X loads hit the staged tile the way real segments do.
template <int G, int P, int RW, int NW, bool DEEP>
__global__ void __launch_bounds__(NW * 32, 1) probe_segment_kernel(float* out, int reps, int L, int nseg,
                                                                   const unsigned char* grec, const int4* ghdr)
{
    constexpr int T = 32 * P;
    extern __shared__ __align__(16) unsigned char sm[];
    float* xt = reinterpret_cast<float*>(sm);
    for (int i = threadIdx.x; i < 64 * T; i += blockDim.x) xt[i] = 1.0f + (i % 977) * 1e-3f;
    unsigned char* recs = sm + 64 * T * 4;
    const int rbytes = nseg * L * alcs::record_bytes(G);
    for (int i = threadIdx.x; i < rbytes / 16; i += blockDim.x) reinterpret_cast<int4*>(recs)[i] = reinterpret_cast<const int4*>(grec)[i];
    int4* hdr = reinterpret_cast<int4*>(recs + rbytes);
    for (int i = threadIdx.x; i < nseg; i += blockDim.x) hdr[i] = ghdr[i];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned char* xs = sm + lane * 16;
    float2 acc[RW][G][P / 2];
#pragma unroll
    for (int s = 0; s < RW; ++s)
#pragma unroll
        for (int j = 0; j < G; ++j)
#pragma unroll
            for (int e = 0; e < P / 2; ++e) acc[s][j][e] = make_float2(0.f, 0.f);
    int seg = (warp * 7) % nseg;
    for (int r = 0; r < reps; ++r) {
#pragma unroll
        for (int s = 0; s < RW; ++s) {
            seg = seg + 1 < nseg ? seg + 1 : 0;
            const int4 hd = hdr[seg];
            if (hd.w > 0) alcs::consume_segment<float, G, P, DEEP>(acc[s], xs, recs + hd.x * 16, hd.w, hd.y, hd.z);
        }
    }
    float sum = 0;
#pragma unroll
    for (int s = 0; s < RW; ++s)
#pragma unroll
        for (int j = 0; j < G; ++j)
#pragma unroll
            for (int e = 0; e < P / 2; ++e) sum += acc[s][j][e].x + acc[s][j][e].y;
    out[blockIdx.x * blockDim.x + threadIdx.x] = sum;
}

struct ProbeEnv {
    int sms = 0;
    double peak = 0;          // SMs x 128 lanes x 2 x maximum SM clock, FLOP/s
    float* out = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    ~ProbeEnv()
    {
        if (out) cudaFree(out);
        if (e0) cudaEventDestroy(e0);
        if (e1) cudaEventDestroy(e1);
    }
};

int probe_env(ProbeEnv& env)
{
    int dev = 0, khz = 0;
    PROBE_CUDA(cudaGetDevice(&dev));
    PROBE_CUDA(cudaDeviceGetAttribute(&env.sms, cudaDevAttrMultiProcessorCount, dev));
    PROBE_CUDA(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
    env.peak = (double)env.sms * 128.0 * 2.0 * khz * 1e3;
    PROBE_CUDA(cudaMalloc(&env.out, (size_t)env.sms * 1024 * sizeof(float)));
    PROBE_CUDA(cudaEventCreate(&env.e0));
    PROBE_CUDA(cudaEventCreate(&env.e1));
    return ALCS_OK;
}

// Best of three timed launches after one warm-up; `launch` enqueues the kernel on st.
template <typename F>
int time_launch(ProbeEnv& env, cudaStream_t st, F launch, double* ms_out)
{
    float best = 1e30f;
    for (int i = 0; i < 4; ++i) {
        PROBE_CUDA(cudaEventRecord(env.e0, st));
        launch();
        PROBE_CUDA(cudaGetLastError());
        PROBE_CUDA(cudaEventRecord(env.e1, st));
        PROBE_CUDA(cudaEventSynchronize(env.e1));
        float ms = 0;
        PROBE_CUDA(cudaEventElapsedTime(&ms, env.e0, env.e1));
        if (i > 0 && ms < best) best = ms;
    }
    *ms_out = best;
    return ALCS_OK;
}

template <int G, int P, int RW, int NW, bool DEEP>
int run_segment_probe(int L, cudaStream_t st, alcs_probe_result* res)
{
    ProbeEnv env;
    int rc = probe_env(env);
    if (rc) return rc;
    const int REC = alcs::record_bytes(G);
    const int T = 32 * P;
    const int budget = 200 * 1024 - 64 * T * 4;
    int nseg = budget / (L * REC + 16);
    if (nseg > 4096) nseg = 4096;
    if (nseg < 1) return ALCS_ERR_SHAPE;
    std::vector<unsigned char> rec((size_t)nseg * L * REC);
    std::vector<int4> hdr(nseg);
    unsigned state = 12345;
    auto rnd = [&]() { state = state * 1664525u + 1013904223u; return (int)((state >> 10) % 64); };
    for (int s = 0; s < nseg; ++s) {
        hdr[s] = make_int4(s * L * REC / 16, rnd(), rnd(), L);
        for (int i = 0; i < L; ++i) {
            unsigned char* r = &rec[((size_t)s * L + i) * REC];
            const int h[4] = {rnd(), rnd(), 0, 0};
            std::memcpy(r, h, G == 1 ? 8 : 16);
            float w[2 * G];
            for (int j = 0; j < 2 * G; ++j) w[j] = 1e-3f * (j + 1);
            std::memcpy(r + (G == 1 ? 8 : 16), w, sizeof w);
        }
    }
    unsigned char* drec = nullptr;
    int4* dhdr = nullptr;
    PROBE_CUDA(cudaMalloc(&drec, rec.size()));
    cudaError_t e = cudaMalloc(&dhdr, hdr.size() * sizeof(int4));
    if (e == cudaSuccess) e = cudaMemcpyAsync(drec, rec.data(), rec.size(), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dhdr, hdr.data(), hdr.size() * sizeof(int4), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    const size_t smem = (size_t)64 * T * 4 + rec.size() + hdr.size() * sizeof(int4);
    auto kern = probe_segment_kernel<G, P, RW, NW, DEEP>;
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaFuncAttributes fa{};
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, kern);
    double ms = 0;
    const int reps = 40000 / L / RW + 1;
    if (e == cudaSuccess) {
        rc = time_launch(env, st, [&]() { kern<<<env.sms, NW * 32, smem, st>>>(env.out, reps, L, nseg, drec, dhdr); }, &ms);
    }
    cudaFree(drec);
    cudaFree(dhdr);
    if (e != cudaSuccess) {
        alcs::set_cuda_error_text(cudaGetErrorString(e));
        (void)cudaGetLastError();
        return ALCS_ERR_CUDA;
    }
    if (rc) return rc;
    const double flop = 2.0 * (double)env.sms * NW * reps * RW * L * 2.0 * G * T;
    res->ms = ms;
    res->tflops = flop / (ms * 1e-3) / 1e12;
    res->frac_of_fp32_peak = flop / (ms * 1e-3) / env.peak;
    res->registers = fa.numRegs;
    res->spill_bytes = (int)fa.localSizeBytes;
    return ALCS_OK;
}

}  // namespace

extern "C" {

ALCS_API int alcs_probe_fma_peak(int packed, alcs_probe_result* out, void* cuda_stream)
{
    if (!out || (packed != 0 && packed != 1)) return ALCS_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof *out);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ProbeEnv env;
    int rc = probe_env(env);
    if (rc) return rc;
    const int iters = 20000;
    double ms = 0;
    cudaFuncAttributes fa{};
    if (packed) {
        PROBE_CUDA(cudaFuncGetAttributes(&fa, probe_ffma2_kernel));
        rc = time_launch(env, st, [&]() { probe_ffma2_kernel<<<env.sms, 512, 0, st>>>(env.out, iters, 1.0001f, 0.5f); }, &ms);
    } else {
        PROBE_CUDA(cudaFuncGetAttributes(&fa, probe_ffma_kernel));
        rc = time_launch(env, st, [&]() { probe_ffma_kernel<<<env.sms, 512, 0, st>>>(env.out, iters, 1.0001f, 0.5f); }, &ms);
    }
    if (rc) return rc;
    const double flop = 2.0 * (packed ? 2.0 : 1.0) * (double)env.sms * 512 * 32.0 * iters;
    out->ms = ms;
    out->tflops = flop / (ms * 1e-3) / 1e12;
    out->frac_of_fp32_peak = flop / (ms * 1e-3) / env.peak;
    out->registers = fa.numRegs;
    out->spill_bytes = (int)fa.localSizeBytes;
    return ALCS_OK;
}

ALCS_API int alcs_probe_lds(int bytes_per_lane, int uniform, double* cycles_per_instruction, void* cuda_stream)
{
    if (!cycles_per_instruction || (uniform != 0 && uniform != 1)) return ALCS_ERR_INVALID_ARG;
    if (bytes_per_lane != 4 && bytes_per_lane != 8 && bytes_per_lane != 16) return ALCS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ProbeEnv env;
    int rc = probe_env(env);
    if (rc) return rc;
    int dev = 0, khz = 0;
    PROBE_CUDA(cudaGetDevice(&dev));
    PROBE_CUDA(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
    const int iters = 20000;
    const size_t smem = 65536;
    double ms = 0;
#define ALCS_LDS_CASE(W, U)                                                                                              \
    if (bytes_per_lane == W && uniform == (U ? 1 : 0)) {                                                                   \
        PROBE_CUDA(cudaFuncSetAttribute(probe_lds_kernel<W, U>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        rc = time_launch(env, st, [&]() { probe_lds_kernel<W, U><<<env.sms, 512, smem, st>>>(env.out, iters); }, &ms);    \
    }
    ALCS_LDS_CASE(16, false) ALCS_LDS_CASE(16, true) ALCS_LDS_CASE(8, false) ALCS_LDS_CASE(8, true)
    ALCS_LDS_CASE(4, false) ALCS_LDS_CASE(4, true)
#undef ALCS_LDS_CASE
    if (rc) return rc;
    const double instr_per_sm = 16.0 * iters * 16;        // 16 warps x iters x 16 loads
    *cycles_per_instruction = ms * 1e-3 * khz * 1e3 / instr_per_sm;
    return ALCS_OK;
}

ALCS_API int alcs_probe_segment_loop(int g, int pixels_per_lane, int rows_per_warp, int warps, int deep,
                                     int pairs_per_segment, alcs_probe_result* out, void* cuda_stream)
{
    if (!out || pairs_per_segment < 1 || pairs_per_segment > 256) return ALCS_ERR_INVALID_ARG;
    std::memset(out, 0, sizeof *out);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
#define ALCS_SEG_CASE(G, P, RW, NW, DEEP)                                                             \
    if (g == G && pixels_per_lane == P && rows_per_warp == RW && warps == NW && (deep != 0) == DEEP) \
        return run_segment_probe<G, P, RW, NW, DEEP>(pairs_per_segment, st, out);
    ALCS_SEG_CASE(4, 8, 2, 16, false)
    ALCS_SEG_CASE(4, 8, 2, 16, true)
    ALCS_SEG_CASE(4, 8, 2, 12, false)
    ALCS_SEG_CASE(4, 8, 2, 12, true)
    ALCS_SEG_CASE(4, 8, 2, 8, true)
    ALCS_SEG_CASE(4, 8, 1, 16, false)
    ALCS_SEG_CASE(4, 16, 1, 16, false)
    ALCS_SEG_CASE(4, 16, 1, 12, true)
    ALCS_SEG_CASE(4, 4, 4, 16, false)
    ALCS_SEG_CASE(1, 8, 2, 16, false)
    ALCS_SEG_CASE(8, 4, 2, 16, false)
    ALCS_SEG_CASE(16, 4, 1, 16, false)
#undef ALCS_SEG_CASE
    return ALCS_ERR_UNSUPPORTED;
}

}  // extern "C"
