// Tensor-core flavour of the sparse pointwise convolution for fp16 weights and activations
// (paper, Section 3.2.2: one block = g consecutive output channels sharing one input channel).
//
// Sixteen kept blocks of one block row form a dense 16 x g weight tile; multiplied with the 16
// input-channel rows they select, it is a real dense contraction D[16 pixels][8 channels] +=
// A[16 pixels][16 channels] * B[16 channels][8 channels] (mma.sync m16n8k16, fp32 accumulate).
// The 16 channel rows are GATHERED: ldmatrix takes one shared-memory address per 8-pixel row, so
// every lane passes the row of the column it is responsible for.  That is why this path uses the
// warp-level MMA and not tcgen05, whose shared-memory operand descriptors can only describe rows
// at a fixed stride.
//
// The staging ring, the producers and the hand-over are those of the CUDA-core kernel; the tile
// rows carry 16 bytes of padding so that rows whose channel indices differ modulo 8 lie in
// different banks (the schedule orders a segment's blocks accordingly).
#ifndef ALCS_MMA_CUH_
#define ALCS_MMA_CUH_

#include "alcs_kernels.cuh"

namespace alcs {

constexpr int kMmaXPad = 16;      // bytes of padding per channel row of the tile

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr)
                 : "memory");
}

__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// One segment: `steps` step records at `rec` (shared memory), X tile at shared address `xs`
// (already offset by this lane's pixel half).  c[mt][nb] are the accumulator tiles.
template <int G, int P>
__device__ __forceinline__ void consume_steps(float (&c)[2 * P][(G < 8 ? 8 : G) / 8][4], uint32_t xs,
                                              const unsigned char* rec, int steps, int lane)
{
    constexpr int MT = 2 * P;                       // 16-pixel tiles per warp tile
    constexpr int NB = (G < 8 ? 8 : G) / 8;         // 8-channel tiles per block row
    constexpr int REC = 32 + 256 * NB;
    constexpr int ROWB = 32 * P * 2 + kMmaXPad;
    const int my_col = (lane & 7) + ((lane >> 4) << 3);     // which of the step's 16 columns this lane addresses
    const unsigned short* colp = reinterpret_cast<const unsigned short*>(rec) + my_col;
    const uint2* wp = reinterpret_cast<const uint2*>(rec + 32) + lane;

    int col = *colp;
    uint2 b[NB];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) b[nb] = wp[nb * 32];
    for (int s = 0; s < steps; ++s) {
        const uint32_t addr = xs + col * ROWB;
        uint2 bn[NB];
        int coln = col;
        if (s + 1 < steps) {                        // next step's column and weights, ahead of use
            coln = *(colp + (s + 1) * (REC / 2));
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) bn[nb] = wp[(s + 1) * (REC / 8) + nb * 32];
        } else {
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) bn[nb] = b[nb];
        }
        uint32_t a[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) ldmatrix_x4_trans(addr + mt * 32, a[mt]);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) mma_m16n8k16(c[mt][nb], a[mt], b[nb].x, b[nb].y);
        col = coln;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) b[nb] = bn[nb];
    }
}

__device__ __forceinline__ void stmatrix_x4_trans(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};\n"
                 :
                 : "r"(addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
                 : "memory");
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// GR = 1: all NW consumer warps work on the same item.  GR = 2: two groups of NW/2 warps take the
// items of the thread block alternately, so that one group's multiply phase (shared-memory bound)
// runs while the other group is in its epilogue (store bound) and the producers stream ahead for
// both; each group has its own half of the ring's stages and barriers.
template <int G, int P, int RW, int NW, int NPW, int MINB, int GR>
__global__ void __launch_bounds__((NW + NPW) * 32, MINB) spconv1x1_mma_kernel(const ConvArgs a)
{
    static_assert(P == 4 || P == 8, "a lane stores runs of 4 or 8 pixels");
    static_assert(GR == 1 || (GR == 2 && NW % 2 == 0), "one or two consumer groups");
    constexpr int NWG = NW / GR;                      // consumer warps per group
    constexpr int T = 32 * P;
    constexpr int MT = 2 * P;
    constexpr int GP = G < 8 ? 8 : G;
    constexpr int NB = GP / 8;
    constexpr int VG = (P * 2 >= 16) ? 8 : P;         // pixels per lane and store vector
    constexpr int NG = P / VG;
    constexpr int SCRB = T * 2 + 16;                  // bytes per channel row of the epilogue scratch (fp16)

    extern __shared__ __align__(16) unsigned char smem[];   // [full[8] | empty[8] | ring | epilogue scratch]

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int S = a.stages;
    const uint32_t smem_u32 = (uint32_t)__cvta_generic_to_shared(smem);

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32 + 8 * s, a.bulk ? 1 : 32 * NPW);
            mbar_init(smem_u32 + 8 * kMaxStages + 8 * s, NWG);
        }
    }
    __syncthreads();
    grid_dep_launch();

    if (warp >= NW) {   // ---- producer warps ------------------------------------------------
        const int pw = warp - NW;
        if (a.bulk) {
            produce_bulk<__half, G, P, kMmaXPad, GR>(a, smem, lane, pw, NPW);
            return;
        }
        switch (a.ld_bytes) {
            case 16: produce<__half, G, P, 16, kMmaXPad, GR>(a, smem, lane, pw, NPW); break;
            case 8: produce<__half, G, P, 8, kMmaXPad, GR>(a, smem, lane, pw, NPW); break;
            case 4: produce<__half, G, P, 4, kMmaXPad, GR>(a, smem, lane, pw, NPW); break;
            default: produce<__half, G, P, 2, kMmaXPad, GR>(a, smem, lane, pw, NPW); break;
        }
        return;
    }

    // ---- consumer warps ---------------------------------------------------------------------
    const unsigned char* ring = smem + 16 * kMaxStages;
    const uint32_t scr_off = 16 * kMaxStages + S * a.stage_bytes + warp * (8 * SCRB);
    const unsigned char* scratch = smem + scr_off;
    const int items = a.n_tiles * a.n_rg;
    const int gid = lane >> 2, tig = lane & 3;
    const int grp = warp / NWG, wg = warp - grp * NWG;
    int kk = 0;
    int turn = 0;

    const int SG = S / GR;                  // stages of this group's half of the ring
    for (int item = blockIdx.x; item < items; item += gridDim.x, turn ^= 1) {
        if (GR == 2 && turn != grp) continue;       // the other group's item
        const int tile = item / a.n_rg;
        const int rg = item - tile * a.n_rg;
        const int q0 = tile * T;

        int lrow[RW], rowid[RW];
        float2 bz[RW][NB];          // bias of the two channels this lane holds in an accumulator tile
#pragma unroll
        for (int s = 0; s < RW; ++s) {
            lrow[s] = s * NWG + ((s & 1) ? NWG - 1 - wg : wg);
            rowid[s] = lrow[s] < a.rpg ? __ldg(a.rowmap + rg * a.rpg + lrow[s]) : -1;
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                const int co = rowid[s] * G + nb * 8 + 2 * tig;
                const bool in0 = rowid[s] >= 0 && a.bias && nb * 8 + 2 * tig < G && co < a.cout;
                const bool in1 = rowid[s] >= 0 && a.bias && nb * 8 + 2 * tig + 1 < G && co + 1 < a.cout;
                bz[s][nb].x = in0 ? __ldg(a.bias + co) : 0.0f;
                bz[s][nb].y = in1 ? __ldg(a.bias + co + 1) : 0.0f;
            }
        }

        float c[RW][MT][NB][4];
#pragma unroll
        for (int s = 0; s < RW; ++s)
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int nb = 0; nb < NB; ++nb)
#pragma unroll
                    for (int e = 0; e < 4; ++e) c[s][mt][nb][e] = 0.0f;

        for (int k = 0; k < a.nch; ++k, ++kk) {
            const int st = grp * SG + kk % SG;
            if (!mbar_wait(smem_u32 + 8 * st, (kk / SG) & 1)) {
                if (lane == 0) atomicExch(a.err, kErrFullWait);
                return;
            }
            const unsigned char* stage = ring + st * a.stage_bytes;
            const uint32_t xs = smem_u32 + 16 * kMaxStages + st * a.stage_bytes + ((lane >> 3) & 1) * 16;
            const unsigned char* recs = stage + a.off_rec;
            const int4* roff = reinterpret_cast<const int4*>(stage + a.off_rowoff);
#pragma unroll
            for (int s = 0; s < RW; ++s) {
                if (lrow[s] >= a.rpg) continue;
                const int4 hd = roff[lrow[s]];     // {segment start, steps, -, -}
                if (hd.y > 0) consume_steps<G, P>(c[s], xs, recs + hd.x * 16, hd.y, lane);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32 + 8 * kMaxStages + 8 * st);
        }

        grid_dep_wait();
        if (a.y_f32) {
            // ---- fp32 output: straight from the accumulator tiles.  A lane holds (pixel gid, channels
            // 2*tig, 2*tig+1) and (pixel gid + 8, same channels) of every 16-pixel tile; the 8 lanes
            // with one tig write 8 consecutive pixels = one 32-byte sector per channel.
            float* ybase = static_cast<float*>(a.y);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int q = q0 + mt * 16 + hf * 8 + gid;
                    if (q >= a.q_total) continue;
                    const int nn = q / a.hw;
                    const int pp = q - nn * a.hw;
                    if (pp >= a.hwy) continue;
                    float* yp = ybase + (size_t)nn * a.cout * a.hwy + pp;
#pragma unroll
                    for (int s = 0; s < RW; ++s) {
                        if (rowid[s] < 0) continue;
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int j = nb * 8 + 2 * tig + e;
                                const int co = rowid[s] * G + j;
                                if (j >= G || co >= a.cout) continue;
                                float v = c[s][mt][nb][2 * hf + e] + (e ? bz[s][nb].y : bz[s][nb].x);
                                if (a.res) v += __ldg(static_cast<const float*>(a.res) + (yp - ybase) + (size_t)co * a.hwy);
                                if (a.relu) v = fmaxf(v, 0.0f);
                                yp[(size_t)co * a.hwy] = v;
                            }
                        }
                    }
                }
            }
        } else {
            // ---- fp16 output: bias and ReLU on the accumulator tiles, then a transposing matrix store
            // into a warp-private scratch tile [8 channels][T pixels], from which every lane reads runs
            // of consecutive pixels of one channel for 16-byte (or 8-byte) global stores.
            __half* ybase = static_cast<__half*>(a.y);
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
            const uint32_t st_addr = smem_u32 + scr_off + (lane & 7) * SCRB + (lane >> 3) * 16;
            const __half2 zero2 = __floats2half2_rn(0.0f, 0.0f);
#pragma unroll
            for (int s = 0; s < RW; ++s) {
                if (rowid[s] < 0) continue;
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    __syncwarp();
                    const __half* rbase = static_cast<const __half*>(a.res);
                    if (rbase) {
                        // The residual takes the way of the output in reverse: every lane copies runs of
                        // consecutive pixels of one channel into the scratch tile, and a transposing matrix
                        // load hands each lane the values at its accumulator positions, so that the sum is
                        // formed in fp32 and rounded once.
#pragma unroll 2
                        for (int j = 0; j < 8; ++j) {
                            const int co = rowid[s] * G + nb * 8 + j;
                            const bool have = nb * 8 + j < G && co < a.cout;
#pragma unroll
                            for (int gi = 0; gi < NG; ++gi) {
                                unsigned char* wp = const_cast<unsigned char*>(scratch) + j * SCRB + (gi * (32 * VG) + lane * VG) * 2;
                                __half* hw16 = reinterpret_cast<__half*>(wp);
                                if (have && a.st_vec && yok[gi]) {
                                    const __half* src = rbase + yoff[gi] + (size_t)co * a.hwy;
                                    if constexpr (VG == 8) *reinterpret_cast<uint4*>(wp) = __ldg(reinterpret_cast<const uint4*>(src));
                                    else *reinterpret_cast<uint2*>(wp) = __ldg(reinterpret_cast<const uint2*>(src));
                                } else if (!a.st_vec && a.st_grp == 1) {
                                    // the run lies in one image (padded rows are a multiple of VG long); its
                                    // pixels p >= hwy exist only as padding of the repacked X
                                    const int nreal = (have && yok[gi]) ? a.hwy - yp[gi] : 0;
                                    const __half* src = rbase + yoff[gi] + (size_t)co * a.hwy;
                                    if (nreal >= VG && (reinterpret_cast<uintptr_t>(src) & (2 * VG - 1)) == 0) {
                                        if constexpr (VG == 8) *reinterpret_cast<uint4*>(wp) = __ldg(reinterpret_cast<const uint4*>(src));
                                        else *reinterpret_cast<uint2*>(wp) = __ldg(reinterpret_cast<const uint2*>(src));
                                    } else {
#pragma unroll
                                        for (int t = 0; t < VG; ++t) hw16[t] = t < nreal ? __ldg(src + t) : __float2half_rn(0.0f);
                                    }
                                } else {
                                    int nn = yn[gi], pp = yp[gi];
#pragma unroll
                                    for (int t = 0; t < VG; ++t) {
                                        while (pp >= a.hw) { pp -= a.hw; ++nn; }
                                        const bool in = have && !a.st_vec && q0 + gi * (32 * VG) + lane * VG + t < a.q_total && pp < a.hwy;
                                        hw16[t] = in ? __ldg(rbase + ((size_t)nn * a.cout + co) * a.hwy + pp) : __float2half_rn(0.0f);
                                        ++pp;
                                    }
                                }
                            }
                        }
                        __syncwarp();
                    }
#pragma unroll
                    for (int mp = 0; mp < MT / 2; ++mp) {
                        uint32_t r[4];
                        float2 rs[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
                        if (rbase) {
                            uint32_t q[4];
                            ldmatrix_x4_trans(st_addr + mp * 64, q);
#pragma unroll
                            for (int i = 0; i < 4; ++i) rs[i] = __half22float2(*reinterpret_cast<const __half2*>(&q[i]));
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {       // tiles 2*mp and 2*mp+1, pixel halves 0 and 1
                            const float* cc = c[s][2 * mp + (i >> 1)][nb];
                            r[i] = pack_half2(cc[2 * (i & 1)] + bz[s][nb].x + rs[i].x, cc[2 * (i & 1) + 1] + bz[s][nb].y + rs[i].y);
                            if (a.relu) {
                                const __half2 h = __hmax2(*reinterpret_cast<const __half2*>(&r[i]), zero2);
                                r[i] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                        }
                        stmatrix_x4_trans(st_addr + mp * 64, r[0], r[1], r[2], r[3]);
                    }
                    __syncwarp();
                    if (a.st_grp == 2) {
                        // element-wise stores: lane l of pass k writes pixel k*32 + l of the tile, so that a
                        // warp's store covers consecutive addresses wherever the pixels lie in one image
#pragma unroll 1
                        for (int k = 0; k < P; ++k) {
                            const int q = q0 + k * 32 + lane;
                            const int nn = q / a.hw;
                            const int pp = q - nn * a.hw;
                            if (q >= a.q_total || pp >= a.hwy) continue;
                            __half* dst = ybase + (size_t)nn * a.cout * a.hwy + pp;
                            const __half* hp = reinterpret_cast<const __half*>(scratch) + k * 32 + lane;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int co = rowid[s] * G + nb * 8 + j;
                                if (nb * 8 + j < G && co < a.cout) dst[(size_t)co * a.hwy] = hp[j * (SCRB / 2)];
                            }
                        }
                        continue;
                    }
#pragma unroll 2
                    for (int j = 0; j < 8; ++j) {
                        const int co = rowid[s] * G + nb * 8 + j;
                        if (nb * 8 + j >= G || co >= a.cout) continue;
#pragma unroll
                        for (int gi = 0; gi < NG; ++gi) {
                            const unsigned char* rp = scratch + j * SCRB + (gi * (32 * VG) + lane * VG) * 2;
                            if (a.st_vec) {
                                if (!yok[gi]) continue;
                                __half* dst = ybase + yoff[gi] + (size_t)co * a.hwy;
                                if constexpr (VG == 8) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(rp);
                                else *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(rp);
                            } else if (a.st_grp == 1) {
                                // the run lies in one image: one vector store where all its pixels are real
                                // and the address allows it (two halves for a 16-byte run on an 8-byte
                                // boundary), single elements otherwise
                                if (!yok[gi]) continue;
                                __half* dst = ybase + yoff[gi] + (size_t)co * a.hwy;
                                const int nreal = a.hwy - yp[gi];
                                const uintptr_t ad = reinterpret_cast<uintptr_t>(dst);
                                if (nreal >= VG && (ad & (2 * VG - 1)) == 0) {
                                    if constexpr (VG == 8) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(rp);
                                    else *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(rp);
                                } else if (VG == 8 && nreal >= VG && (ad & 7) == 0) {
                                    *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(rp);
                                    *reinterpret_cast<uint2*>(dst + 4) = *reinterpret_cast<const uint2*>(rp + 8);
                                } else {
                                    const __half* hp = reinterpret_cast<const __half*>(rp);
#pragma unroll
                                    for (int t = 0; t < VG; ++t)
                                        if (t < nreal) dst[t] = hp[t];
                                }
                            } else {
                                // element by element: the run may cross into the next image, and pixels
                                // p >= hwy exist only as padding of the repacked X
                                const __half* hp = reinterpret_cast<const __half*>(rp);
                                int nn = yn[gi], pp = yp[gi];
#pragma unroll
                                for (int t = 0; t < VG; ++t) {
                                    while (pp >= a.hw) { pp -= a.hw; ++nn; }
                                    if (q0 + gi * (32 * VG) + lane * VG + t < a.q_total && pp < a.hwy)
                                        ybase[((size_t)nn * a.cout + co) * a.hwy + pp] = hp[t];
                                    ++pp;
                                }
                            }
                        }
                    }
                }
            }
        }
    }
}

#define ALCS_MMA_VARIANT(G, P, RW, NW, NPW, MINB, GR) \
    {1, G, P, RW, NW, MINB, NPW, (const void*)&spconv1x1_mma_kernel<G, P, RW, NW, NPW, MINB, GR>, 1, GR}

}  // namespace alcs

#endif  // ALCS_MMA_CUH_
