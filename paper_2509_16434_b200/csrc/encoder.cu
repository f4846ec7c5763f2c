// Encoder forward/backward: the direct first convolution (C_in = 1), pooling, the small
// element-wise kernels, and the orchestration of the implicit GEMMs of the deeper layers.
#include "common.cuh"
#include "gemm.cuh"

// -------------------------------------------------------------------- conv1 ----

// First layer (C_in = 1): too shallow a reduction (k*k) for a tensor-core tile, and bound by
// HBM (reads one fp16 frame, writes C1 bf16 maps).  One thread per output pixel; the k*k
// patch sits in registers, the weights (as the bf16 shadow rounds them) in shared memory.
// With STAGE the 16-byte chunks of a warp's 32 pixels pass through a swizzled shared-memory
// buffer so that every store instruction of the warp writes 512 contiguous bytes (C1 / 8 a
// power of two); without it each thread stores its own pixel.
template <int KS, bool STAGE>
__global__ void __launch_bounds__(128) conv1_fwd_kernel(const __half *__restrict__ depth,
                                                        const bf16 *__restrict__ W, const float *__restrict__ bias,
                                                        bf16 *__restrict__ out, uint32_t *__restrict__ bits,
                                                        int rows, int Hi, int Wi, int Ho, int Wo, int C1) {
    extern __shared__ __align__(16) float sm[];  // w[tap][co], then bias[co], then (STAGE) 4 warps x 32 pixels x C1 bf16
    float *w = sm, *bs = sm + KS * KS * C1;
    for (int i = threadIdx.x; i < KS * KS * C1; i += blockDim.x) {
        const int co = i % C1, tap = i / C1;
        w[i] = bf2f(W[co * KS * KS + tap]);
    }
    for (int i = threadIdx.x; i < C1; i += blockDim.x) bs[i] = bias[i];
    __syncthreads();
    const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long M = (long long)rows * Ho * Wo;
    const bool live = m < M;
    constexpr int P = KS / 2;
    float x[KS * KS];
    if (live) {
        const int ow = (int)(m % Wo);
        const long long t = m / Wo;
        const int oh = (int)(t % Ho);
        const __half *img = depth + (t / Ho) * Hi * Wi;
#pragma unroll
        for (int kh = 0; kh < KS; ++kh)
#pragma unroll
            for (int kw = 0; kw < KS; ++kw) {
                const int ih = 2 * oh + kh - P, iw = 2 * ow + kw - P;
                x[kh * KS + kw] = (ih >= 0 && ih < Hi && iw >= 0 && iw < Wi) ? __half2float(img[ih * Wi + iw]) : 0.f;
            }
    } else {
#pragma unroll
        for (int i = 0; i < KS * KS; ++i) x[i] = 0.f;
    }
    const int CH = C1 >> 3;  // 16-byte chunks per pixel
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint4 *stage = reinterpret_cast<uint4 *>(bs + C1) + (size_t)warp * 32 * CH;
    const int sh = CH == 8 ? 0 : (CH == 4 ? 1 : (CH == 2 ? 2 : 3));
    uint4 *o = reinterpret_cast<uint4 *>(out + m * C1);
    uint32_t gate = 0;  // ReLU gate bits of the current 32 channels
    for (int c8 = 0; c8 < C1; c8 += 8) {
        float acc[8];
        {
            const float4 b0 = *reinterpret_cast<const float4 *>(bs + c8), b1 = *reinterpret_cast<const float4 *>(bs + c8 + 4);
            acc[0] = b0.x; acc[1] = b0.y; acc[2] = b0.z; acc[3] = b0.w;
            acc[4] = b1.x; acc[5] = b1.y; acc[6] = b1.z; acc[7] = b1.w;
        }
#pragma unroll
        for (int tap = 0; tap < KS * KS; ++tap) {
            const float4 w0 = *reinterpret_cast<const float4 *>(w + tap * C1 + c8);
            const float4 w1 = *reinterpret_cast<const float4 *>(w + tap * C1 + c8 + 4);
            const float xv = x[tap];
            acc[0] = fmaf(w0.x, xv, acc[0]); acc[1] = fmaf(w0.y, xv, acc[1]);
            acc[2] = fmaf(w0.z, xv, acc[2]); acc[3] = fmaf(w0.w, xv, acc[3]);
            acc[4] = fmaf(w1.x, xv, acc[4]); acc[5] = fmaf(w1.y, xv, acc[5]);
            acc[6] = fmaf(w1.z, xv, acc[6]); acc[7] = fmaf(w1.w, xv, acc[7]);
        }
        __nv_bfloat162 p[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) p[j] = __floats2bfloat162_rn(fmaxf(acc[2 * j], 0.f), fmaxf(acc[2 * j + 1], 0.f));
        if (bits) {
#pragma unroll
            for (int j = 0; j < 4; ++j) gate = gate_bits_add(gate, *reinterpret_cast<uint32_t *>(&p[j]), ((c8 & 31) >> 1) + j);
            if ((c8 & 31) == 24) {
                if (live) bits[m * (C1 >> 5) + (c8 >> 5)] = gate;
                gate = 0;
            }
        }
        if (STAGE) stage[lane * CH + ((c8 >> 3) ^ ((lane >> sh) & (CH - 1)))] = *reinterpret_cast<uint4 *>(p);
        else if (live) o[c8 >> 3] = *reinterpret_cast<uint4 *>(p);
    }
    if (STAGE) {
        __syncwarp();
        const long long mw = m - lane;  // first pixel of this warp
        for (int i = lane; i < 32 * CH; i += 32) {
            const int px = i / CH, phys = i - px * CH;
            const int chunk = phys ^ ((px >> sh) & (CH - 1));
            if (mw + px < M) reinterpret_cast<uint4 *>(out + (mw + px) * C1)[chunk] = stage[i];
        }
    }
}

// dW1[co][tap] += sum_m dZ1[m][co] * x(m, tap);  db1[co] += sum_m dZ1[m][co].
// A lane owns CPT consecutive channels; C1 / CPT lanes share a pixel and a warp walks 32 CPT / C1
// pixels per step through a contiguous range of output pixels: the gradient rows are read once,
// coalesced, 2 CPT bytes per lane, while a pixel's k*k input taps are one broadcast load each, paid
// once per CPT * (k*k + 1) multiply-adds.  All loads of a trip (U steps) are issued before the first
// use.  Every lane keeps CPT (k*k + 1) accumulators (the last of each channel is the bias gradient);
// they are folded across the pixel slots of a warp by shuffles, across warps through shared memory,
// and left as this block's partial sums in part[blockIdx.x][C1 k*k (dW order) | C1 (db)], which
// sum_partials_kernel adds up in block order.  C1 / CPT must be a power of two <= 32.
template <int KS, int CPT, int U>
__global__ void __launch_bounds__(128) conv1_wgrad_kernel(const __half *__restrict__ depth,
                                                          const bf16 *__restrict__ dZ, float *__restrict__ part,
                                                          int rows, int Hi, int Wi, int Ho,
                                                          int Wo, int C1, long long px_per_warp) {
    constexpr int K2 = KS * KS, P = KS / 2;
    extern __shared__ float sm[];  // [4 warps][C1 * (K2 + 1)]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lpp = C1 / CPT;      // lanes per pixel
    const int ppi = 32 / lpp;      // pixels per step
    const int cq = lane % lpp, ps = lane / lpp;
    float acc[CPT][K2 + 1];
#pragma unroll
    for (int c = 0; c < CPT; ++c)
#pragma unroll
        for (int t = 0; t <= K2; ++t) acc[c][t] = 0.f;
    const long long M = (long long)rows * Ho * Wo;
    const long long gw = (long long)blockIdx.x * 4 + warp;
    long long m = gw * px_per_warp + ps;
    const long long m_end = min(M, (gw + 1) * px_per_warp);
    if (m < m_end) {
        int ow = (int)(m % Wo);
        long long t = m / Wo;
        int oh = (int)(t % Ho);
        long long b = t / Ho;
        for (; m < m_end; m += (long long)U * ppi) {
            uint32_t dzr[U][CPT / 2];
            __half xr[U][K2];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long mu = m + (long long)u * ppi;
                const bool live = mu < m_end;
                const bf16 *zp = dZ + mu * C1 + cq * CPT;
                if (CPT == 8) {
                    const uint4 r = live ? __ldcs(reinterpret_cast<const uint4 *>(zp)) : make_uint4(0, 0, 0, 0);
                    dzr[u][0] = r.x; dzr[u][1 % (CPT / 2)] = r.y; dzr[u][2 % (CPT / 2)] = r.z; dzr[u][3 % (CPT / 2)] = r.w;
                } else if (CPT == 4) {
                    const uint2 r = live ? __ldcs(reinterpret_cast<const uint2 *>(zp)) : make_uint2(0, 0);
                    dzr[u][0] = r.x; dzr[u][1 % (CPT / 2)] = r.y;
                } else {
                    dzr[u][0] = live ? __ldcs(reinterpret_cast<const uint32_t *>(zp)) : 0u;
                }
                const __half *img = depth + b * Hi * Wi;
#pragma unroll
                for (int kh = 0; kh < KS; ++kh) {
                    const int ih = 2 * oh + kh - P;
#pragma unroll
                    for (int kw = 0; kw < KS; ++kw) {
                        const int iw = 2 * ow + kw - P;
                        const bool in = live && ih >= 0 && ih < Hi && iw >= 0 && iw < Wi;
                        xr[u][kh * KS + kw] = in ? __ldg(img + ih * Wi + iw) : __float2half_rn(0.f);
                    }
                }
                ow += ppi;
                while (ow >= Wo) {
                    ow -= Wo;
                    if (++oh == Ho) { oh = 0; ++b; }
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float xv[K2];
#pragma unroll
                for (int k = 0; k < K2; ++k) xv[k] = __half2float(xr[u][k]);
#pragma unroll
                for (int c2 = 0; c2 < CPT / 2; ++c2) {
                    const float2 dz = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&dzr[u][c2]));
#pragma unroll
                    for (int k = 0; k < K2; ++k) {
                        acc[2 * c2][k] = fmaf(dz.x, xv[k], acc[2 * c2][k]);
                        acc[2 * c2 + 1][k] = fmaf(dz.y, xv[k], acc[2 * c2 + 1][k]);
                    }
                    acc[2 * c2][K2] += dz.x;
                    acc[2 * c2 + 1][K2] += dz.y;
                }
            }
        }
    }
    // fold the pixel slots of the warp (lanes that differ in bits >= log2(lpp))
#pragma unroll
    for (int c = 0; c < CPT; ++c)
#pragma unroll
        for (int t = 0; t <= K2; ++t) {
            float v = acc[c][t];
            for (int o = lpp; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            acc[c][t] = v;
        }
    const int per = C1 * (K2 + 1);
    if (lane < lpp) {
#pragma unroll
        for (int c = 0; c < CPT; ++c)
#pragma unroll
            for (int t = 0; t <= K2; ++t) sm[warp * per + (cq * CPT + c) * (K2 + 1) + t] = acc[c][t];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < per; i += 128) {
        float v = 0.f;
        for (int w = 0; w < 4; ++w) v += sm[w * per + i];
        const int co = i / (K2 + 1), t = i % (K2 + 1);
        part[(size_t)blockIdx.x * per + (t < K2 ? co * K2 + t : C1 * K2 + co)] = v;
    }
}

// The same reduction on the tensor cores (mma.sync m16n8k16, bf16): per 16 output pixels a warp forms
// D[tap][co] += X^T[tap][px] dZ[px][co] with the pixel index as K (32 pixels, one per lane, per trip).  The patch tile X
// and the 16 x C1 gradient tile go through per-warp shared memory and come back as fragments with ldmatrix.trans.
// A lane fetches its pixel's window as aligned pairs of fp16 frame pixels (32-bit loads) and converts each pair to bf16
// in three instructions; the tap axis is laid out as (window row, pair, element of the pair) -- one element per row lies
// outside the window and its row of D is dropped -- followed by a column of ones whose product is the bias gradient,
// zero padded to TP.  About 3 instructions per pixel and channel-independent instead of C1 (k*k + 1) / 32 multiply-adds
// plus their loads: the kernel becomes a stream over dZ.  C1 must be a multiple of 16 and the frame width even.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int KS, int NB>  // NB = C1 / 8 column blocks
__global__ void __launch_bounds__(256) conv1_wgrad_mma_kernel(const __half *__restrict__ depth,
                                                              const bf16 *__restrict__ dZ, float *__restrict__ part,
                                                              int rows, int Hi, int Wi,
                                                              int Ho, int Wo, long long px_per_warp) {
    constexpr int K2 = KS * KS, P = KS / 2, ODD = P & 1, NP = (KS + ODD + 1) / 2, KW = KS * NP;
    constexpr int TP = (2 * KW + 1 + 15) / 16 * 16, MB = TP / 16, C1 = NB * 8;
    constexpr int PX = 32;  // pixels per trip: one per lane, two K = 16 steps of the MMA
    constexpr int kXBytes = PX * TP * 2, kZBytes = PX * C1 * 2;
    extern __shared__ __align__(16) uint8_t smw[];  // per warp: X tile [32 px][TP], dZ tile [32 px][C1]; later the reduction
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t *xs = smw + (size_t)warp * (kXBytes + kZBytes), *zs = xs + kXBytes;
    const uint32_t xs_a = (uint32_t)__cvta_generic_to_shared(xs), zs_a = (uint32_t)__cvta_generic_to_shared(zs);
    float acc[MB][NB][4];
#pragma unroll
    for (int i = 0; i < MB; ++i)
#pragma unroll
        for (int j = 0; j < NB; ++j)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[i][j][q] = 0.f;
    const long long M = (long long)rows * Ho * Wo;
    const long long gw = (long long)blockIdx.x * 8 + warp;
    long long m0 = gw * px_per_warp;                       // px_per_warp is a multiple of 32
    const long long m_end = min(M, m0 + px_per_warp);
    int ow = 0, oh = 0;  // this lane's pixel m0 + lane
    long long b = 0;
    if (m0 < m_end) {
        const long long m = m0 + lane;
        ow = (int)(m % Wo);
        const long long t = m / Wo;
        oh = (int)(t % Ho);
        b = t / Ho;
    }
    const int d_oh = PX / Wo, d_ow = PX % Wo;  // 32 pixels further (Wo >= 1)
    constexpr int ZP = PX * C1 / 8 / 32;       // 16-byte pieces of the gradient tile per lane
    uint4 xreg[TP / 8], zreg[ZP];
    // Loads of the tile that starts at pixel mt into registers; they are issued one trip ahead, so that their
    // latency overlaps the previous tile's MMAs.
    const int Wh = Wi >> 1;  // 32-bit words per frame row
    auto prefetch = [&](long long mt) {
        const bool live = mt + lane < m_end;
        // every load is issued, from a clamped address where its pixel pair lies outside the frame, before the first
        // conversion: the loads of a trip are then in flight together
        const uint32_t *img = reinterpret_cast<const uint32_t *>(depth) + (live ? b : 0) * Hi * Wh;
        uint32_t wv[TP / 2], raw[KW];
        const int pw0 = ow - (P + ODD) / 2;
        uint32_t okm = 0;
#pragma unroll
        for (int kh = 0; kh < KS; ++kh) {
            const int ih = 2 * oh + kh - P;
            const bool rok = live && (unsigned)ih < (unsigned)Hi;
            const uint32_t *row = img + (rok ? ih : 0) * Wh;
#pragma unroll
            for (int q = 0; q < NP; ++q) {
                const int pw = pw0 + q;
                const bool ok = rok && (unsigned)pw < (unsigned)Wh;
                raw[kh * NP + q] = __ldg(row + (ok ? pw : 0));
                okm |= (ok ? 1u : 0u) << (kh * NP + q);
            }
        }
#pragma unroll
        for (int k = 0; k < TP / 2; ++k) wv[k] = 0u;
#pragma unroll
        for (int k = 0; k < KW; ++k) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&raw[k]));
            wv[k] = (okm >> k) & 1u ? pack_bf16x2(f.x, f.y) : 0u;
        }
        if (live) wv[KW] = 0x00003F80u;  // (1.0, 0) as bf16: the bias-gradient column
#pragma unroll
        for (int c = 0; c < TP / 8; ++c) xreg[c] = make_uint4(wv[4 * c], wv[4 * c + 1], wv[4 * c + 2], wv[4 * c + 3]);
#pragma unroll
        for (int z = 0; z < ZP; ++z) {
            const int i = lane + 32 * z;
            zreg[z] = make_uint4(0, 0, 0, 0);
            if (mt + i / (C1 / 8) < m_end) zreg[z] = __ldcs(reinterpret_cast<const uint4 *>(dZ + mt * C1) + i);
        }
    };
    if (m0 < m_end) prefetch(m0);
    for (; m0 < m_end; m0 += PX) {
#pragma unroll
        for (int c = 0; c < TP / 8; ++c) *reinterpret_cast<uint4 *>(xs + lane * (TP * 2) + c * 16) = xreg[c];
#pragma unroll
        for (int z = 0; z < ZP; ++z) reinterpret_cast<uint4 *>(zs)[lane + 32 * z] = zreg[z];
        __syncwarp();
        ow += d_ow;
        if (ow >= Wo) { ow -= Wo; ++oh; }
        oh += d_oh;
        while (oh >= Ho) { oh -= Ho; ++b; }
        if (m0 + PX < m_end) prefetch(m0 + PX);
        // ---- fragments and MMAs, 16 pixels per K step
#pragma unroll
        for (int ks = 0; ks < PX / 16; ++ks) {
            uint32_t af[MB][4];
            const int mi = lane >> 3, r = lane & 7;
#pragma unroll
            for (int i = 0; i < MB; ++i) {
                // matrices: (taps 16i..+7, px 0-7), (taps 16i+8.., px 0-7), (taps 16i.., px 8-15), (taps 16i+8.., px 8-15)
                const uint32_t addr =
                    xs_a + (uint32_t)((16 * ks + r + (mi >= 2 ? 8 : 0)) * (TP * 2) + (16 * i + (mi & 1) * 8) * 2);
                ldmatrix_x4_trans(addr, af[i][0], af[i][1], af[i][2], af[i][3]);
            }
#pragma unroll
            for (int j = 0; j < NB; j += 2) {
                // matrices: (px 0-7, co 8j..), (px 8-15, co 8j..), (px 0-7, co 8j+8..), (px 8-15, co 8j+8..)
                const uint32_t addr =
                    zs_a + (uint32_t)((16 * ks + r + (mi & 1) * 8) * (C1 * 2) + (8 * j + (mi >> 1) * 8) * 2);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(addr, b0, b1, b2, b3);
#pragma unroll
                for (int i = 0; i < MB; ++i) {
                    mma_bf16_16816(acc[i][j], af[i][0], af[i][1], af[i][2], af[i][3], b0, b1);
                    mma_bf16_16816(acc[i][j + 1], af[i][0], af[i][1], af[i][2], af[i][3], b2, b3);
                }
            }
        }
        __syncwarp();
    }
    // ---- block reduction: D element (tap = 16 i + g (+8), co = 8 j + 2 c (+1)) -> [TP][C1] floats per warp
    __syncthreads();
    float *red = reinterpret_cast<float *>(smw);
    constexpr int per = TP * C1;
    {
        const int g = lane >> 2, c = lane & 3;
        float *mine = red + (size_t)warp * per;
#pragma unroll
        for (int i = 0; i < MB; ++i)
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                mine[(16 * i + g) * C1 + 8 * j + 2 * c] = acc[i][j][0];
                mine[(16 * i + g) * C1 + 8 * j + 2 * c + 1] = acc[i][j][1];
                mine[(16 * i + g + 8) * C1 + 8 * j + 2 * c] = acc[i][j][2];
                mine[(16 * i + g + 8) * C1 + 8 * j + 2 * c + 1] = acc[i][j][3];
            }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < (2 * KW + 1) * C1; i += 256) {
        const int t = i / C1, co = i - t * C1;   // row t of D: element t & 1 of pair (t >> 1) % NP of window row (t >> 1) / NP
        const int kh = (t >> 1) / NP, kw = 2 * ((t >> 1) - kh * NP) + (t & 1) - ODD;
        if (t < 2 * KW && (kw < 0 || kw >= KS)) continue;
        float v = 0.f;
        for (int w = 0; w < 8; ++w) v += red[(size_t)w * per + i];
        // this block's partial sums, [C1 k*k (dW order) | C1 (db)]; sum_partials_kernel adds the blocks up in order
        part[(size_t)blockIdx.x * (C1 * (K2 + 1)) + (t < 2 * KW ? co * K2 + kh * KS + kw : C1 * K2 + co)] = v;
    }
}

// ------------------------------------------------------------- small kernels ----

// One thread per 32 channels of a pixel: the ReLU gate (act > 0) as a bit mask, channel c at bit
// gate_bit_of_channel(c).
__global__ void __launch_bounds__(256) relu_bits_kernel(const bf16 *__restrict__ act, uint32_t *__restrict__ bits,
                                                        long long words) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= words) return;
    const uint4 *p = reinterpret_cast<const uint4 *>(act + i * 32);
    uint32_t w = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint4 r = p[j];
        const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&r);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float2 f = __bfloat1622float2(h2[q]);
            w |= (f.x > 0.f ? 1u : 0u) << (j * 4 + q);
            w |= (f.y > 0.f ? 1u : 0u) << (16 + j * 4 + q);
        }
    }
    bits[i] = w;
}

int relu_bits(const bf16 *act, uint32_t *bits, long long M, int C, cudaStream_t st) {
    if (C % 32 != 0) return PPO_ERR_UNSUPPORTED;
    const long long words = M * (C / 32);
    if (words <= 0) return PPO_OK;
    relu_bits_kernel<<<ppo_cdiv(words, 256), 256, 0, st>>>(act, bits, words);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}


// h0[b] = [mean over pixels of act[b][px][c], proprio[b]] as bf16.  One warp per row b; a lane
// owns 8 channels at a time so that every pixel is read with 128-bit loads.
__global__ void __launch_bounds__(256) pool_concat_kernel(const bf16 *__restrict__ act,
                                                          const float *__restrict__ proprio, bf16 *__restrict__ h0,
                                                          int rows, int npx, int C, int P) {
    const int b = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= rows) return;
    const float inv = 1.f / (float)npx;
    const bf16 *base = act + (size_t)b * npx * C;
    bf16 *out = h0 + (size_t)b * (C + P);
    for (int c8 = lane * 8; c8 < C; c8 += 256) {
        float s[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) s[i] = 0.f;
        for (int px = 0; px < npx; ++px) {
            const uint4 raw = *reinterpret_cast<const uint4 *>(base + (size_t)px * C + c8);
            const __nv_bfloat162 *p2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(p2[i]);
                s[2 * i] += f.x;
                s[2 * i + 1] += f.y;
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) out[c8 + i] = __float2bfloat16_rn(s[i] * inv);
    }
    for (int j = lane; j < P; j += 32) out[C + j] = __float2bfloat16_rn(proprio[(size_t)b * P + j]);
}

// dact[b][px][c] = dh0[b][c] / npx where act > 0, else 0; 8 channels per thread.
__global__ void __launch_bounds__(256) unpool_kernel(const float *__restrict__ dh0, const bf16 *__restrict__ act,
                                                     bf16 *__restrict__ dact, long long total8, int npx, int C,
                                                     int ld_h0) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total8) return;
    const int c8n = C >> 3;
    const int c8 = (int)(i % c8n) * 8;
    const long long b = i / ((long long)npx * c8n);
    const float inv = 1.f / (float)npx;
    const float4 g0 = *reinterpret_cast<const float4 *>(dh0 + b * ld_h0 + c8);
    const float4 g1 = *reinterpret_cast<const float4 *>(dh0 + b * ld_h0 + c8 + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const uint4 raw = *reinterpret_cast<const uint4 *>(act + i * 8);
    const __nv_bfloat162 *a2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
    __nv_bfloat162 o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 f = __bfloat1622float2(a2[k]);
        o[k] = __floats2bfloat162_rn(f.x > 0.f ? g[2 * k] * inv : 0.f, f.y > 0.f ? g[2 * k + 1] * inv : 0.f);
    }
    *reinterpret_cast<uint4 *>(dact + i * 8) = *reinterpret_cast<uint4 *>(o);
}

// Head gradient as a bf16 GEMM operand: [rows][16] = [dmean (A), dvalue, zeros].
__global__ void __launch_bounds__(256) pack_dout_kernel(const float *__restrict__ dmean,
                                                        const float *__restrict__ dvalue, bf16 *__restrict__ out,
                                                        int rows, int A) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * 16) return;
    const int r = i / 16, j = i % 16;
    float v = 0.f;
    if (j < A) v = dmean[(size_t)r * A + j];
    else if (j == A) v = dvalue[r];
    out[i] = __float2bfloat16_rn(v);
}

#define PPO_TRY(expr)                 \
    do {                              \
        int _s = (expr);              \
        if (_s != PPO_OK) return _s;  \
    } while (0)

// dst[i] (i < nA: dstA[i], else dstB[i - nA]) += part[0][i] + part[1][i] + ... in that order: the second stage of the
// reductions whose blocks leave partial sums instead of adding to the result with atomics (reproducible results).
__global__ void __launch_bounds__(256) sum_partials_kernel(const float *__restrict__ part, int nparts, int nA,
                                                           float *__restrict__ dstA, int nB, float *__restrict__ dstB) {
    // 32 results per block; eight threads share a result, thread j adding the partials b = j, j + 8, ... in order, and
    // the eight sums are added in the order of j: fixed, whatever the launch.
    __shared__ float sh[8][32];
    const int o = threadIdx.x & 31, j = threadIdx.x >> 5;
    const int i = blockIdx.x * 32 + o;
    const int n = nA + nB;
    part += (size_t)blockIdx.y * nparts * n;  // blockIdx.y: one of several independent reductions of nA results (nB = 0)
    dstA += (size_t)blockIdx.y * nA;
    float acc = 0.f;
    if (i < n)
        for (int b = j; b < nparts; b += 8) acc += part[(size_t)b * n + i];
    sh[j][o] = acc;
    __syncthreads();
    if (j == 0 && i < n) {
        float v = sh[0][o];
#pragma unroll
        for (int q = 1; q < 8; ++q) v += sh[q][o];
        if (i < nA) dstA[i] += v;
        else dstB[i - nA] += v;
    }
}

static int sum_partials(const float *part, int nparts, int nA, float *dstA, int nB, float *dstB, cudaStream_t st,
                        int slabs = 1) {
    sum_partials_kernel<<<dim3(ppo_cdiv(nA + nB, 32), slabs), 256, 0, st>>>(part, nparts, nA, dstA, nB, dstB);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

// part[block][n] = sum over this block's rows m of dZ[m][n]  (bias gradients, first stage), N a multiple of 8.  Threads
// walk (row, 8-column chunk) pairs with 128-bit loads; threads that share a chunk are folded through shared memory.
__global__ void __launch_bounds__(256) colsum_kernel(const bf16 *__restrict__ dZ, int ld, long long M, int N,
                                                     float *__restrict__ part) {
    __shared__ float sh[256][9];
    const int chunks = N >> 3;                    // 16-byte chunks per row
    const int rows_per_pass = 256 / chunks;       // whole rows covered by one pass of the block
    const int tc = threadIdx.x % chunks, tr = threadIdx.x / chunks;
    dZ += (size_t)blockIdx.y * N;  // blockIdx.y: slab of N columns of a wider matrix
    part += (size_t)blockIdx.y * gridDim.x * N;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    if (tr < rows_per_pass) {
        for (long long m = (long long)blockIdx.x * rows_per_pass + tr; m < M;
             m += (long long)gridDim.x * rows_per_pass) {
            const uint4 raw = *reinterpret_cast<const uint4 *>(dZ + m * ld + tc * 8);
            const __nv_bfloat162 *p2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(p2[i]);
                acc[2 * i] += f.x;
                acc[2 * i + 1] += f.y;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) sh[threadIdx.x][i] = acc[i];
    __syncthreads();
    if (threadIdx.x < N) {
        const int c = threadIdx.x >> 3, e = threadIdx.x & 7;
        float v = 0.f;
        for (int r = 0; r < rows_per_pass; ++r) v += sh[r * chunks + c][e];
        part[(size_t)blockIdx.x * N + threadIdx.x] = v;
    }
}

// The same first stage for any N <= ld (used for the head, whose 13 columns sit in rows of 16).
__global__ void __launch_bounds__(256) colsum_small_kernel(const bf16 *__restrict__ dZ, int ld, long long M, int N,
                                                           float *__restrict__ part) {
    __shared__ float sh[256];
    for (int n = 0; n < N; ++n) {
        float v = 0.f;
        for (long long m = (long long)blockIdx.x * 256 + threadIdx.x; m < M; m += (long long)gridDim.x * 256)
            v += bf2f(dZ[m * ld + n]);
        sh[threadIdx.x] = v;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
            __syncthreads();
        }
        if (threadIdx.x == 0) part[(size_t)blockIdx.x * N + n] = sh[0];
        __syncthreads();
    }
}

// Wt[ci][tap][co (row stride ld)] = W[co][tap][ci], zero in the padding co >= Co.
__global__ void __launch_bounds__(256) transpose_weights_kernel(const bf16 *__restrict__ W, bf16 *__restrict__ Wt,
                                                                int Co, int taps, int Ci, int ld) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)Ci * taps * ld;
    if (i >= total) return;
    const int co = (int)(i % ld);
    const long long r = i / ld;
    const int tap = (int)(r % taps), ci = (int)(r / taps);
    Wt[i] = (co < Co) ? W[((size_t)co * taps + tap) * Ci + ci] : __float2bfloat16_rn(0.f);
}

// h0[b][E .. E+P) = proprio[b] as bf16 (the embedding occupies the first E columns of a row of ld elements).
__global__ void __launch_bounds__(256) concat_proprio_kernel(const float *__restrict__ proprio, bf16 *__restrict__ h0,
                                                             int rows, int E, int P, int ld) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * P) return;
    const int b = i / P, j = i - b * P;
    h0[(size_t)b * ld + E + j] = __float2bfloat16_rn(proprio[i]);
}

// dz[b][e] = dh0[b][e] where the embedding h0[b][e] is > 0, else 0 (back through its ReLU), as a bf16 GEMM operand.
__global__ void __launch_bounds__(256) embed_dz_kernel(const float *__restrict__ dh0, const bf16 *__restrict__ h0,
                                                       bf16 *__restrict__ dz, int rows, int E, int ld) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * E) return;
    const int b = i / E, e = i - b * E;
    const float v = bf2f(h0[(size_t)b * ld + e]) > 0.f ? dh0[(size_t)b * ld + e] : 0.f;
    dz[i] = __float2bfloat16_rn(v);
}

// Backward of the layer normalisation of one conv layer, in place on the gradient: d [M][C] holds dL/d(gamma xhat + beta)
// (already zero where the ReLU was off) and leaves dL/dz,
//   t = gamma d,  dz = rstd (t - mean_c(t) - xhat mean_c(t xhat)),
// and every block leaves its partial sums of dgamma = sum d xhat and dbeta = sum d in part[block][2 C].  C / 8 lanes
// share a pixel (8 channels each, one 128-bit access per array), C a power of two in 16 .. 256.
__global__ void __launch_bounds__(256) ln_bwd_kernel(bf16 *__restrict__ d, const bf16 *__restrict__ xhat,
                                                     const float *__restrict__ rstd, const float *__restrict__ gamma,
                                                     long long M, int C, float *__restrict__ part) {
    __shared__ float sh[16][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lpp = C >> 3, ppw = 32 / lpp;
    const int cq = lane % lpp, slot = lane / lpp;
    float gm[8], dg[8], db[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        gm[i] = gamma[cq * 8 + i];
        dg[i] = 0.f;
        db[i] = 0.f;
    }
    const float inv_c = 1.f / (float)C;
    for (long long px0 = ((long long)blockIdx.x * 8 + warp) * ppw; px0 < M; px0 += (long long)gridDim.x * 8 * ppw) {
        const long long px = px0 + slot;
        const bool live = px < M;
        float dv[8], xv[8], t[8];
        uint4 rd = make_uint4(0, 0, 0, 0), rx = make_uint4(0, 0, 0, 0);
        float rs = 0.f;
        if (live) {
            rd = *reinterpret_cast<const uint4 *>(d + px * C + cq * 8);
            rx = *reinterpret_cast<const uint4 *>(xhat + px * C + cq * 8);
            rs = rstd[px];
        }
        const __nv_bfloat162 *d2 = reinterpret_cast<const __nv_bfloat162 *>(&rd);
        const __nv_bfloat162 *x2 = reinterpret_cast<const __nv_bfloat162 *>(&rx);
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 a = __bfloat1622float2(d2[i]), b = __bfloat1622float2(x2[i]);
            dv[2 * i] = a.x; dv[2 * i + 1] = a.y;
            xv[2 * i] = b.x; xv[2 * i + 1] = b.y;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            t[i] = gm[i] * dv[i];
            s1 += t[i];
            s2 += t[i] * xv[i];
            dg[i] += dv[i] * xv[i];
            db[i] += dv[i];
        }
        for (int o = 1; o < lpp; o <<= 1) {  // the lanes of a pixel are adjacent
            s1 += __shfl_xor_sync(0xffffffffu, s1, o);
            s2 += __shfl_xor_sync(0xffffffffu, s2, o);
        }
        const float m1 = s1 * inv_c, m2 = s2 * inv_c;
        if (live) {
            uint4 o4;
            o4.x = pack_bf16x2(rs * (t[0] - m1 - xv[0] * m2), rs * (t[1] - m1 - xv[1] * m2));
            o4.y = pack_bf16x2(rs * (t[2] - m1 - xv[2] * m2), rs * (t[3] - m1 - xv[3] * m2));
            o4.z = pack_bf16x2(rs * (t[4] - m1 - xv[4] * m2), rs * (t[5] - m1 - xv[5] * m2));
            o4.w = pack_bf16x2(rs * (t[6] - m1 - xv[6] * m2), rs * (t[7] - m1 - xv[7] * m2));
            *reinterpret_cast<uint4 *>(d + px * C + cq * 8) = o4;
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        sh[i][threadIdx.x] = dg[i];
        sh[8 + i][threadIdx.x] = db[i];
    }
    __syncthreads();
    // channel ch of kind k (0: dgamma, 1: dbeta): the threads whose lane % lpp == ch / 8, in thread order
    for (int o = threadIdx.x; o < 2 * C; o += 256) {
        const int k = o / C, ch = o - k * C, q = ch >> 3, e = k * 8 + (ch & 7);
        float v = 0.f;
        for (int tdx = q; tdx < 256; tdx += lpp) v += sh[e][tdx];
        part[(size_t)blockIdx.x * 2 * C + o] = v;
    }
}

// ------------------------------------------------------------ recurrent trunk ----

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + __expf(-x)); }

// State the first step of a sequence starts from: h_prev[0] = bf16(h_init), c_prev[0] = c_init (rows of one step, Be x H).
__global__ void __launch_bounds__(256) lstm_init_kernel(const float *__restrict__ h_init, const float *__restrict__ c_init,
                                                        bf16 *__restrict__ hprev, float *__restrict__ cprev, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    hprev[i] = __float2bfloat16_rn(h_init[i]);
    cprev[i] = c_init[i];
}

// One time step of one LSTM layer for Be envs, element-wise part: gate pre-activations = xg + hg + b,
//   (i, f, g, o) = (sigmoid, sigmoid, tanh, sigmoid)(.),  c = f c_prev + i g,  h = o tanh(c).
// Keeps the gate activations and c for the backward pass, writes h as bf16 (the operand of the next contractions) and,
// unless this is the last step, the state the next step starts from: (h, c) or zeros where done != 0.
__global__ void __launch_bounds__(256) lstm_cell_fwd_kernel(const float *__restrict__ xg, const float *__restrict__ hg,
                                                            const float *__restrict__ bias, const float *__restrict__ cprev,
                                                            const uint8_t *__restrict__ done, float *__restrict__ gates,
                                                            float *__restrict__ c, bf16 *__restrict__ h,
                                                            bf16 *__restrict__ hprev_next, float *__restrict__ cprev_next,
                                                            int Be, int H) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Be * H) return;
    const int e = i / H, j = i - e * H;
    const size_t g0 = (size_t)e * 4 * H + j;
    const float gi = sigmoidf_(xg[g0] + hg[g0] + bias[j]);
    const float gf = sigmoidf_(xg[g0 + H] + hg[g0 + H] + bias[H + j]);
    const float gg = tanhf(xg[g0 + 2 * H] + hg[g0 + 2 * H] + bias[2 * H + j]);
    const float go = sigmoidf_(xg[g0 + 3 * H] + hg[g0 + 3 * H] + bias[3 * H + j]);
    const float cv = gf * cprev[i] + gi * gg;
    const float hv = go * tanhf(cv);
    gates[g0] = gi;
    gates[g0 + H] = gf;
    gates[g0 + 2 * H] = gg;
    gates[g0 + 3 * H] = go;
    c[i] = cv;
    const bf16 hb = __float2bfloat16_rn(hv);
    h[i] = hb;
    if (hprev_next) {
        const bool reset = done[e] != 0;
        hprev_next[i] = reset ? __float2bfloat16_rn(0.f) : hb;
        cprev_next[i] = reset ? 0.f : cv;
    }
}

// The same step backwards.  dtop: gradient w.r.t. this step's h from above; dhc, dcc: gradients w.r.t. the state the
// NEXT step started from (raw: they count only where this step's done flag is clear; dhc arrives as nsplit partial
// products, Be * H floats apart, that are added in order).  Writes the gradient of the gate pre-activations as bf16 (a
// GEMM operand) and the raw gradient of c_prev; the raw gradient of h_prev comes out of the GEMM dg W_h that follows.
// last != 0: no step follows, nothing is carried.
__global__ void __launch_bounds__(256) lstm_cell_bwd_kernel(const float *__restrict__ dtop, const float *__restrict__ dhc,
                                                            float *__restrict__ dcc, const uint8_t *__restrict__ done,
                                                            const float *__restrict__ gates, const float *__restrict__ c,
                                                            const float *__restrict__ cprev, bf16 *__restrict__ dg,
                                                            int Be, int H, int last, int nsplit) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Be * H) return;
    const int e = i / H, j = i - e * H;
    const size_t g0 = (size_t)e * 4 * H + j;
    const bool carry = !last && done[e] == 0;
    float dhn = 0.f;
    if (carry)
        for (int s = 0; s < nsplit; ++s) dhn += dhc[(size_t)s * Be * H + i];
    const float dh = dtop[i] + dhn;
    const float gi = gates[g0], gf = gates[g0 + H], gg = gates[g0 + 2 * H], go = gates[g0 + 3 * H];
    const float tc = tanhf(c[i]);
    const float dc = (carry ? dcc[i] : 0.f) + dh * go * (1.f - tc * tc);
    dg[g0] = __float2bfloat16_rn(dc * gg * gi * (1.f - gi));
    dg[g0 + H] = __float2bfloat16_rn(dc * cprev[i] * gf * (1.f - gf));
    dg[g0 + 2 * H] = __float2bfloat16_rn(dc * gi * (1.f - gg * gg));
    dg[g0 + 3 * H] = __float2bfloat16_rn(dh * tc * go * (1.f - go));
    dcc[i] = dc * gf;
}

// ------------------------------------------------------------ orchestration ----

static ConvGeom conv_geom(const ppo_model *m, int l, int rows) {  // conv layer l in 1..L
    ConvGeom g;
    g.B = rows;
    g.Hi = m->Hs[l - 1];
    g.Wi = m->Ws[l - 1];
    g.Ci = m->Cs[l - 1];
    g.Ho = m->Hs[l];
    g.Wo = m->Ws[l];
    g.Co = m->Cs[l];
    g.k = m->d.conv_k[l - 1];
    g.pad = g.k / 2;
    return g;
}

static ConvGeom fc_geom(int rows, int in, int out) {
    ConvGeom g;
    g.B = rows;
    g.Hi = g.Wi = g.Ho = g.Wo = 1;
    g.Ci = in;
    g.Co = out;
    g.k = 1;
    g.pad = 0;
    return g;
}

static int run_fwd(const ppo_model *m, const ConvGeom &g, const bf16 *X, const bf16 *W, const FwdEpilogue &e,
                   cudaStream_t st) {
    int s = tma_gemm_fwd(g, X, W, e, ppo_device_status_ptr(), st);  // writes e.out_bits itself
    if (s != PPO_ERR_UNSUPPORTED) return s;
    s = tc_gemm_fwd(g, X, W, e, ppo_device_status_ptr(), st);
    if (s == PPO_OK && e.out_bits) s = relu_bits(e.out, e.out_bits, g.M(), g.Co, st);
    return s;
}

static int run_dgrad(const ppo_model *m, const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *W, const bf16 *Wt,
                     int wt_ld, const bf16 *Wc, const DgradEpilogue &e, cudaStream_t st) {
    const int s = tma_gemm_dgrad(g, dY, ldy, Wt, wt_ld, Wc, e, ppo_device_status_ptr(), st);
    if (s != PPO_ERR_UNSUPPORTED) return s;
    return tc_gemm_dgrad(g, dY, ldy, Wt, wt_ld, e, ppo_device_status_ptr(), st);
}

static int run_colsum(const bf16 *dZ, int ld, long long M, int N, float *db, float *part, cudaStream_t st);

// Weight and bias gradients of the layer whose weight matrix is tensor ti.  The TMA kernel of a convolution sums
// the bias gradient on the tensor core on its way; everything else reduces dY in a pass of its own.
static int run_wgrad(const ppo_model *m, int ti, const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X,
                     cudaStream_t st, bool with_bias = true) {
    float *dW = m->grad + m->tensors[ti].off, *db = with_bias ? m->grad + m->tensors[ti + 1].off : nullptr;
    float *part = m->wg_part[ti];
    const size_t cap = m->wg_cap[ti];
    const bool conv = g.k > 1;
    int s = tma_gemm_wgrad(g, dY, ldy, X, dW, conv ? db : nullptr, part, cap, ppo_device_status_ptr(), st);
    if (s == PPO_OK && conv) return s;
    if (s == PPO_ERR_UNSUPPORTED && conv) s = tma_gemm_wgrad(g, dY, ldy, X, dW, nullptr, part, cap, ppo_device_status_ptr(), st);
    if (s == PPO_ERR_UNSUPPORTED) s = tc_gemm_wgrad(g, dY, ldy, X, dW, part, cap, ppo_device_status_ptr(), st);
    if (s != PPO_OK || !with_bias) return s;
    return run_colsum(dY, ldy, g.M(), g.Co, db, m->cs_part[ti], st);
}

// Blocks a column sum of M rows is cut into (first stage), at most 4 per SM.
static int colsum_blocks(long long M, long long rows_per_block) {
    int blocks = ppo_cdiv(M, rows_per_block);
    const int cap = ppo_num_sms() * 4;
    return blocks > cap ? cap : (blocks < 1 ? 1 : blocks);
}

// db[n] += sum_m dZ[m][n] in two stages; `part` holds 4 x SMs x max(N, 16) floats.
static int run_colsum(const bf16 *dZ, int ld, long long M, int N, float *db, float *part, cudaStream_t st) {
    if (N % 8 == 0 && N <= 256 && ld % 8 == 0) {
        const int rows_per_pass = 256 / (N / 8);
        const int blocks = colsum_blocks(M, (long long)rows_per_pass * 8);
        colsum_kernel<<<blocks, 256, 0, st>>>(dZ, ld, M, N, part);
        PPO_LAUNCH_CHECK();
        return sum_partials(part, blocks, N, db, 0, nullptr, st);
    }
    if (N > 256 && N % 256 == 0) {
        // wide layers: slabs of 256 columns along the grid's second axis
        const int blocks = colsum_blocks(M, 64);
        colsum_kernel<<<dim3(blocks, N / 256), 256, 0, st>>>(dZ, ld, M, 256, part);
        PPO_LAUNCH_CHECK();
        return sum_partials(part, blocks, 256, db, 0, nullptr, st, N / 256);
    }
    int blocks = ppo_cdiv(M, 2048);
    blocks = blocks > 64 ? 64 : (blocks < 1 ? 1 : blocks);
    colsum_small_kernel<<<blocks, 256, 0, st>>>(dZ, ld, M, N, part);
    PPO_LAUNCH_CHECK();
    return sum_partials(part, blocks, N, db, 0, nullptr, st);
}


static int check_rows(const ppo_model *m, const ppo_minibatch *mb, int row0, int rows) {
    if (!m || !mb) return PPO_ERR_INVALID_ARG;
    if (!m->master) return PPO_ERR_STATE;
    if (row0 < 0 || rows <= 0 || row0 + rows > mb->B || rows > m->mbmax) return PPO_ERR_SHAPE;
    if (!mb->depth_f16 || !mb->proprio) return PPO_ERR_INVALID_ARG;
    return PPO_OK;
}

// Input of FC layer l (1..F; F + 1 is the head): the layer below, and for the first one h_0 or, behind a recurrent
// trunk, the top LSTM layer's outputs.
static const bf16 *fc_input(const ppo_model *m, int l) {
    if (l > 1) return m->h[l - 1];
    return m->d.n_lstm > 0 ? m->lstm_hs[m->d.n_lstm - 1] : m->h[0];
}
static int fc_input_width(const ppo_model *m, int l) { return l > 1 ? m->hw[l - 1] : m->fc_in_w; }

static int wt_ld_of(int Co) { return (Co + 7) / 8 * 8; }

// out [rows][N] (fp32, row stride N) = A [rows][K] (bf16, row stride lda) . Wn [N][K]^T: the plain product behind every
// contraction of the recurrent trunk, through the flat (1x1-image) input-gradient GEMM.
// ksplit > 1: the reduction is cut into that many slabs and `out` receives their partial products one after another
// (rows * N floats each), for the reader to add in order.
static int gemm_nt_f32(const ppo_model *m, int rows, int N, int K, const bf16 *A, int lda, const bf16 *Wn, float *out,
                       cudaStream_t st, int ksplit = 1) {
    ConvGeom g = fc_geom(rows, N, K);
    DgradEpilogue e = {nullptr, nullptr, out};
    e.ksplit = ksplit;
    if (ksplit > 1) return tma_gemm_dgrad(g, A, lda, Wn, K, nullptr, e, ppo_device_status_ptr(), st);
    return run_dgrad(m, g, A, lda, Wn, Wn, K, nullptr, e, st);
}

// Forward of the recurrent trunk over the announced sequence (rows = T * Be, time-major): per layer one GEMM for
// W_x x of all rows, then per step the GEMM W_h h_prev and the element-wise cell.
static int lstm_forward(ppo_model *m, int rows, cudaStream_t st) {
    const ppo_model_desc &d = m->d;
    const int T = m->seq_T, Be = m->seq_Be, H = d.lstm_h;
    if (T <= 0 || T * Be != rows || !m->seq_done) return PPO_ERR_STATE;
    for (int l = 0; l < d.n_lstm; ++l) {
        const int in = l == 0 ? m->hw[0] : H, ti = m->ti_lstm[l];
        const bf16 *X = l == 0 ? m->h[0] : m->lstm_hs[l - 1];
        float *cprev = m->lstm_c[l] + (size_t)m->mbmax * H;
        PPO_TRY(gemm_nt_f32(m, rows, 4 * H, in, X, in, m->shadow + m->tensors[ti].off, m->lstm_xg, st));
        lstm_init_kernel<<<ppo_cdiv((long long)Be * H, 256), 256, 0, st>>>(m->seq_h_init + (size_t)l * Be * H,
                                                                          m->seq_c_init + (size_t)l * Be * H,
                                                                          m->lstm_hprev[l], cprev, Be * H);
        PPO_LAUNCH_CHECK();
        for (int t = 0; t < T; ++t) {
            const size_t r0 = (size_t)t * Be;
            PPO_TRY(gemm_nt_f32(m, Be, 4 * H, H, m->lstm_hprev[l] + r0 * H, H, m->shadow + m->tensors[ti + 1].off, m->lstm_hg, st));
            const bool last = t == T - 1;
            lstm_cell_fwd_kernel<<<ppo_cdiv((long long)Be * H, 256), 256, 0, st>>>(
                m->lstm_xg + r0 * 4 * H, m->lstm_hg, m->master + m->tensors[ti + 2].off, cprev + r0 * H, m->seq_done + r0,
                m->lstm_gates[l] + r0 * 4 * H, m->lstm_c[l] + r0 * H, m->lstm_hs[l] + r0 * H,
                last ? nullptr : m->lstm_hprev[l] + (r0 + Be) * H, last ? nullptr : cprev + (r0 + Be) * H, Be, H);
            PPO_LAUNCH_CHECK();
        }
    }
    return PPO_OK;
}

// Back-propagation through time.  In: lstm_dtop = dL/d(top layer's outputs) [rows][H] fp32.  Out: dh0_f32 = dL/dh_0 and
// the gradients of every layer's W_x, W_h and b.
static int lstm_backward(ppo_model *m, int rows, cudaStream_t st) {
    const ppo_model_desc &d = m->d;
    const int T = m->seq_T, Be = m->seq_Be, H = d.lstm_h;
    if (T <= 0 || T * Be != rows || !m->seq_done) return PPO_ERR_STATE;
    for (int l = d.n_lstm - 1; l >= 0; --l) {
        const int in = l == 0 ? m->hw[0] : H, ti = m->ti_lstm[l];
        const bf16 *X = l == 0 ? m->h[0] : m->lstm_hs[l - 1];
        const float *cprev = m->lstm_c[l] + (size_t)m->mbmax * H;
        // dg W_h reduces over 4H columns into few output tiles: with few envs the reduction is cut into four slabs that
        // as many CTAs work on, and the next cell kernel adds their partial products (dhc holds rows * H floats)
        int nsplit = (T >= 4 && Be <= 512) ? 4 : 1;
        for (int t = T - 1; t >= 0; --t) {
            const size_t r0 = (size_t)t * Be;
            lstm_cell_bwd_kernel<<<ppo_cdiv((long long)Be * H, 256), 256, 0, st>>>(
                m->lstm_dtop + r0 * H, m->lstm_dhc, m->lstm_dcc, m->seq_done + r0, m->lstm_gates[l] + r0 * 4 * H,
                m->lstm_c[l] + r0 * H, cprev + r0 * H, m->lstm_dg + r0 * 4 * H, Be, H, t == T - 1 ? 1 : 0, nsplit);
            PPO_LAUNCH_CHECK();
            if (t > 0) {  // raw gradient of the state this step started from: dg W_h
                int s = PPO_ERR_UNSUPPORTED;
                if (nsplit > 1)
                    s = gemm_nt_f32(m, Be, H, 4 * H, m->lstm_dg + r0 * 4 * H, 4 * H, m->wT + m->wT_off[ti + 1], m->lstm_dhc, st, nsplit);
                if (s == PPO_ERR_UNSUPPORTED) {
                    nsplit = 1;
                    s = gemm_nt_f32(m, Be, H, 4 * H, m->lstm_dg + r0 * 4 * H, 4 * H, m->wT + m->wT_off[ti + 1], m->lstm_dhc, st);
                }
                PPO_TRY(s);
            }
        }
        // over all steps at once: the weight gradients, the bias gradient and the gradient of the layer's input
        PPO_TRY(run_wgrad(m, ti, fc_geom(rows, in, 4 * H), m->lstm_dg, 4 * H, X, st, false));
        PPO_TRY(run_wgrad(m, ti + 1, fc_geom(rows, H, 4 * H), m->lstm_dg, 4 * H, m->lstm_hprev[l], st, false));
        PPO_TRY(run_colsum(m->lstm_dg, 4 * H, rows, 4 * H, m->grad + m->tensors[ti + 2].off, m->cs_part[ti], st));
        PPO_TRY(gemm_nt_f32(m, rows, in, 4 * H, m->lstm_dg, 4 * H, m->wT + m->wT_off[ti], l == 0 ? m->dh0_f32 : m->lstm_dtop, st));
    }
    return PPO_OK;
}

extern "C" int ppo_encoder_fwd(ppo_model *m, const ppo_minibatch *mb, int row0, int rows, float *mean, float *value,
                               void *stream) {
    PPO_TRY(check_rows(m, mb, row0, rows));
    if (!mean || !value) return PPO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const ppo_model_desc &d = m->d;
    m->fwd_valid = false;
    {   // conv1
        const __half *depth = static_cast<const __half *>(mb->depth_f16) + (size_t)row0 * d.H * d.W;
        const int C1 = m->Cs[1], KS = d.conv_k[0];
        const long long M = (long long)rows * m->Hs[1] * m->Ws[1];
        const bool norm = d.norm != 0;
        const int tcs = conv1_tc_fwd(depth, m->shadow + m->tensors[0].off, m->master + m->tensors[1].off, m->act[1],
                                     m->abits[1], rows, d.H, d.W, m->Hs[1], m->Ws[1], C1, KS,
                                     norm ? m->master + m->tensors[2].off : nullptr,
                                     norm ? m->master + m->tensors[3].off : nullptr, norm ? m->xhat[1] : nullptr,
                                     norm ? m->rstd[1] : nullptr, ppo_device_status_ptr(), st);
        if (tcs != PPO_OK && (tcs != PPO_ERR_UNSUPPORTED || norm)) return tcs;  // only the tensor-core kernel normalises
        const int CH = C1 / 8;
        const bool stage = CH == 1 || CH == 2 || CH == 4 || CH == 8;
        const size_t smem = (size_t)(KS * KS * C1 + C1) * sizeof(float) + (stage ? (size_t)4 * 32 * C1 * 2 : 0);
        const bf16 *W = m->shadow + m->tensors[0].off;
        const float *bias = m->master + m->tensors[1].off;
        const int blocks = ppo_cdiv(M, 128);
#define PPO_CONV1(KS_)                                                                                              \
    do {                                                                                                            \
        if (stage)                                                                                                  \
            conv1_fwd_kernel<KS_, true><<<blocks, 128, smem, st>>>(depth, W, bias, m->act[1], m->abits[1], rows, d.H, d.W,       \
                                                                   m->Hs[1], m->Ws[1], C1);                         \
        else                                                                                                        \
            conv1_fwd_kernel<KS_, false><<<blocks, 128, smem, st>>>(depth, W, bias, m->act[1], m->abits[1], rows, d.H, d.W,      \
                                                                    m->Hs[1], m->Ws[1], C1);                        \
    } while (0)
        if (tcs == PPO_OK) { /* done on the tensor cores */ }
        else if (KS == 1) PPO_CONV1(1);
        else if (KS == 3) PPO_CONV1(3);
        else if (KS == 5) PPO_CONV1(5);
        else PPO_CONV1(7);
#undef PPO_CONV1
        PPO_LAUNCH_CHECK();
    }
    for (int l = 2; l <= m->L; ++l) {
        ConvGeom g = conv_geom(m, l, rows);
        const int tc = m->ti_conv[l];
        FwdEpilogue e = {m->master + m->tensors[tc + 1].off, 1, m->act[l], nullptr, nullptr, 0};
        e.out_bits = m->abits[l];
        if (d.norm) {
            e.ln_gamma = m->master + m->tensors[tc + 2].off;
            e.ln_beta = m->master + m->tensors[tc + 3].off;
            e.ln_xhat = m->xhat[l];
            e.ln_rstd = m->rstd[l];
        }
        PPO_TRY(run_fwd(m, g, m->act[l - 1], m->shadow + m->tensors[tc].off, e, st));
    }
    if (m->ti_embed >= 0) {
        // flatten -> fully connected -> ReLU into the first E columns of h_0, proprio behind them
        ConvGeom g = fc_geom(rows, m->Hs[m->L] * m->Ws[m->L] * m->Cs[m->L], d.embed);
        FwdEpilogue e = {m->master + m->tensors[m->ti_embed + 1].off, 1, m->h[0], nullptr, nullptr, 0};
        e.ldo = m->hw[0];
        PPO_TRY(run_fwd(m, g, m->act[m->L], m->shadow + m->tensors[m->ti_embed].off, e, st));
        concat_proprio_kernel<<<ppo_cdiv((long long)rows * d.P, 256), 256, 0, st>>>(mb->proprio + (size_t)row0 * d.P, m->h[0],
                                                                                  rows, d.embed, d.P, m->hw[0]);
    } else {
        pool_concat_kernel<<<ppo_cdiv(rows, 8), 256, 0, st>>>(m->act[m->L], mb->proprio + (size_t)row0 * d.P, m->h[0], rows,
                                                              m->Hs[m->L] * m->Ws[m->L], m->Cs[m->L], d.P);
    }
    PPO_LAUNCH_CHECK();
    if (d.n_lstm > 0) PPO_TRY(lstm_forward(m, rows, st));
    int ti = m->ti_fc[1];
    for (int l = 1; l <= m->F; ++l, ti += 2) {
        ConvGeom g = fc_geom(rows, fc_input_width(m, l), m->hw[l]);
        FwdEpilogue e = {m->master + m->tensors[ti + 1].off, 1, m->h[l], nullptr, nullptr, 0};
        PPO_TRY(run_fwd(m, g, fc_input(m, l), m->shadow + m->tensors[ti].off, e, st));
    }
    {
        ConvGeom g = fc_geom(rows, fc_input_width(m, m->F + 1), d.A + 1);
        FwdEpilogue e = {m->master + m->tensors[ti + 1].off, 0, nullptr, mean, value, d.A};
        PPO_TRY(run_fwd(m, g, fc_input(m, m->F + 1), m->shadow + m->tensors[ti].off, e, st));
    }
    m->fwd_valid = true;
    m->last_row0 = row0;
    m->last_rows = rows;
    return PPO_OK;
}

static int refresh_transposed(ppo_model *m, cudaStream_t st) {
    if (m->wT_valid) return PPO_OK;
    for (int l = 2; l <= m->L; ++l) {
        const int Co = m->Cs[l], Ci = m->Cs[l - 1], taps = m->d.conv_k[l - 1] * m->d.conv_k[l - 1];
        const int tc = m->ti_conv[l];
        const long long total = (long long)Ci * taps * wt_ld_of(Co);
        transpose_weights_kernel<<<ppo_cdiv(total, 256), 256, 0, st>>>(m->shadow + m->tensors[tc].off,
                                                                     m->wT + m->wT_off[tc], Co, taps, Ci, wt_ld_of(Co));
        PPO_LAUNCH_CHECK();
        PPO_TRY(tma_dgrad_weights(m->shadow + m->tensors[tc].off, m->wC + m->wC_off[l], Co, m->d.conv_k[l - 1], Ci,
                                  wt_ld_of(Co), st));
    }
    if (m->ti_embed >= 0) {
        const int Ci = m->Hs[m->L] * m->Ws[m->L] * m->Cs[m->L], Co = m->d.embed;
        const long long total = (long long)Ci * wt_ld_of(Co);
        transpose_weights_kernel<<<ppo_cdiv(total, 256), 256, 0, st>>>(m->shadow + m->tensors[m->ti_embed].off,
                                                                     m->wT + m->wT_off[m->ti_embed], Co, 1, Ci, wt_ld_of(Co));
        PPO_LAUNCH_CHECK();
    }
    for (int l = 0; l < m->d.n_lstm; ++l) {
        const int H = m->d.lstm_h, in = l == 0 ? m->hw[0] : H, tl = m->ti_lstm[l];
        transpose_weights_kernel<<<ppo_cdiv((long long)in * 4 * H, 256), 256, 0, st>>>(m->shadow + m->tensors[tl].off,
                                                                                     m->wT + m->wT_off[tl], 4 * H, 1, in, 4 * H);
        PPO_LAUNCH_CHECK();
        transpose_weights_kernel<<<ppo_cdiv((long long)H * 4 * H, 256), 256, 0, st>>>(m->shadow + m->tensors[tl + 1].off,
                                                                                    m->wT + m->wT_off[tl + 1], 4 * H, 1, H, 4 * H);
        PPO_LAUNCH_CHECK();
    }
    int ti = m->ti_fc[1];
    for (int l = 1; l <= m->F + 1; ++l, ti += 2) {
        const int Ci = fc_input_width(m, l), Co = (l <= m->F) ? m->hw[l] : m->d.A + 1;
        const long long total = (long long)Ci * wt_ld_of(Co);
        transpose_weights_kernel<<<ppo_cdiv(total, 256), 256, 0, st>>>(m->shadow + m->tensors[ti].off,
                                                                     m->wT + m->wT_off[ti], Co, 1, Ci, wt_ld_of(Co));
        PPO_LAUNCH_CHECK();
    }
    m->wT_valid = true;
    return PPO_OK;
}

// Second stream and the two events of the fork/join in the backward pass, made on first use.
static int side_stream(ppo_model *m) {
    if (m->side) return PPO_OK;
    cudaStream_t s = nullptr;
    cudaEvent_t ef = nullptr, ej = nullptr;
    if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ef, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ej, cudaEventDisableTiming) != cudaSuccess) {
        if (ej) cudaEventDestroy(ej);
        if (ef) cudaEventDestroy(ef);
        if (s) cudaStreamDestroy(s);
        return PPO_ERR_CUDA;
    }
    m->side = s;  // all three exist, or none is kept
    m->ev_fork = ef;
    m->ev_join = ej;
    return PPO_OK;
}

// conv1: weight and bias gradients only (there is no dgrad into the depth image).
static int conv1_wgrad(ppo_model *m, const ppo_minibatch *mb, int row0, int rows, cudaStream_t st) {
    const ppo_model_desc &d = m->d;
    const __half *depth = static_cast<const __half *>(mb->depth_f16) + (size_t)row0 * d.H * d.W;
    const int C1 = m->Cs[1], KS = d.conv_k[0];
    const long long M = (long long)rows * m->Hs[1] * m->Ws[1];
    if (C1 % 16 == 0 && C1 <= 64 && (KS == 3 || KS == 5) && d.W % 2 == 0 && ppo_aligned(depth, 4)) {
        // tensor-core reduction
        const int TP = KS == 3 ? 16 : 32;
        const size_t tile = (size_t)32 * TP * 2 + (size_t)32 * C1 * 2, redb = (size_t)TP * C1 * sizeof(float);
        const size_t smem = 8 * (tile > redb ? tile : redb);
        int blocks = ppo_cdiv(M, 8 * 16 * 8);
        const int cap = ppo_num_sms() * 4;
        blocks = blocks > cap ? cap : (blocks < 1 ? 1 : blocks);
        long long per_warp = (M + (long long)blocks * 8 - 1) / ((long long)blocks * 8);
        per_warp = (per_warp + 31) / 32 * 32;
        float *dW = m->grad + m->tensors[0].off, *db = m->grad + m->tensors[1].off;
        if ((size_t)blocks * C1 * (KS * KS + 1) > m->c1_cap) return PPO_ERR_SHAPE;
#define PPO_C1W(KS_, NB_)                                                                                    \
    do {                                                                                                     \
        if (smem > 48 * 1024)                                                                                \
            PPO_CUDA_CHECK(cudaFuncSetAttribute(conv1_wgrad_mma_kernel<KS_, NB_>,                            \
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));    \
        conv1_wgrad_mma_kernel<KS_, NB_><<<blocks, 256, smem, st>>>(depth, m->dact[1], m->c1_part, rows, d.H, \
                                                                    d.W, m->Hs[1], m->Ws[1], per_warp);      \
    } while (0)
        const int nb = C1 / 8;
        if (KS == 3 && nb == 2) PPO_C1W(3, 2);
        else if (KS == 3 && nb == 4) PPO_C1W(3, 4);
        else if (KS == 3 && nb == 6) PPO_C1W(3, 6);
        else if (KS == 3 && nb == 8) PPO_C1W(3, 8);
        else if (KS == 5 && nb == 2) PPO_C1W(5, 2);
        else if (KS == 5 && nb == 4) PPO_C1W(5, 4);
        else if (KS == 5 && nb == 6) PPO_C1W(5, 6);
        else PPO_C1W(5, 8);
#undef PPO_C1W
        PPO_LAUNCH_CHECK();
        return sum_partials(m->c1_part, blocks, C1 * KS * KS, dW, C1, db, st);
    }
    const int cpt = KS <= 3 ? 8 : (KS == 5 ? 4 : 2);
    const int lpp = C1 / cpt;
    if (C1 % cpt != 0 || lpp > 32 || (lpp & (lpp - 1)) != 0) return PPO_ERR_UNSUPPORTED;
    const int ppi = 32 / lpp;
    const size_t smem = (size_t)4 * C1 * (KS * KS + 1) * sizeof(float);
    int blocks = ppo_cdiv(M, 4 * 256);
    const int cap = ppo_num_sms() * 6;
    blocks = blocks > cap ? cap : (blocks < 1 ? 1 : blocks);
    long long per_warp = (M + (long long)blocks * 4 - 1) / ((long long)blocks * 4);
    per_warp = (per_warp + ppi - 1) / ppi * ppi;
    float *dW = m->grad + m->tensors[0].off, *db = m->grad + m->tensors[1].off;
    if ((size_t)blocks * C1 * (KS * KS + 1) > m->c1_cap) return PPO_ERR_SHAPE;
#define PPO_CONV1W(KS_, CPT_, U_)                                                                                 \
    conv1_wgrad_kernel<KS_, CPT_, U_><<<blocks, 128, smem, st>>>(depth, m->dact[1], m->c1_part, rows, d.H, d.W,  \
                                                             m->Hs[1], m->Ws[1], C1, per_warp)
    if (smem > 48 * 1024) {
        if (KS == 5) PPO_CUDA_CHECK(cudaFuncSetAttribute(conv1_wgrad_kernel<5, 4, 1>,
                                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (KS == 7) PPO_CUDA_CHECK(cudaFuncSetAttribute(conv1_wgrad_kernel<7, 2, 1>,
                                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    if (KS == 1) PPO_CONV1W(1, 8, 2);
    else if (KS == 3) PPO_CONV1W(3, 8, 2);
    else if (KS == 5) PPO_CONV1W(5, 4, 1);
    else PPO_CONV1W(7, 2, 1);
#undef PPO_CONV1W
    PPO_LAUNCH_CHECK();
    return sum_partials(m->c1_part, blocks, C1 * KS * KS, dW, C1, db, st);
}

extern "C" int ppo_encoder_bwd(ppo_model *m, const ppo_minibatch *mb, int row0, int rows, const float *dmean,
                               const float *dvalue, int accumulate, void *stream) {
    PPO_TRY(check_rows(m, mb, row0, rows));
    if (!dmean || !dvalue) return PPO_ERR_INVALID_ARG;
    if (!m->fwd_valid || m->last_row0 != row0 || m->last_rows != rows) return PPO_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const ppo_model_desc &d = m->d;
    const int L = m->L, F = m->F;
    if (!accumulate)  // everything but the trailing log-sigma slot, which the loss call owns
    {
        PPO_CUDA_CHECK(cudaMemsetAsync(m->grad, 0, (size_t)m->tensors.back().off * sizeof(float), st));
        ppo_count_launches(1);
    }
    PPO_TRY(refresh_transposed(m, st));

    pack_dout_kernel<<<ppo_cdiv((long long)rows * 16, 256), 256, 0, st>>>(dmean, dvalue, m->dh[F + 1], rows, d.A);
    PPO_LAUNCH_CHECK();
    // Weight and bias gradients are leaves of the dependency graph: only the chain of dgrads has to run in order.
    // The leaves of the FC layers (small kernels on a fraction of the SMs) and, further down, conv1's wgrad go to
    // a second stream that forks from the caller's stream whenever the gradient they read is ready and joins it
    // at the end of the call.
    const bool fork = side_stream(m) == PPO_OK;
    cudaStream_t leaf = fork ? m->side : st;
    auto fork_here = [&]() -> int {
        if (!fork) return PPO_OK;
        PPO_CUDA_CHECK(cudaEventRecord(m->ev_fork, st));
        PPO_CUDA_CHECK(cudaStreamWaitEvent(m->side, m->ev_fork, 0));
        return PPO_OK;
    };
    auto join = [&](int status) -> int {
        if (fork) {
            PPO_CUDA_CHECK(cudaEventRecord(m->ev_join, m->side));
            PPO_CUDA_CHECK(cudaStreamWaitEvent(st, m->ev_join, 0));
        }
        return status;
    };
    PPO_TRY(fork_here());
    // head and hidden FC layers, last to first; layer index F+1 is the head
    for (int l = F + 1; l >= 1; --l) {
        const int ti = m->ti_fc[l];
        const int Co = (l <= F) ? m->hw[l] : d.A + 1;
        const int ldy = (l <= F) ? Co : 16;
        ConvGeom g = fc_geom(rows, fc_input_width(m, l), Co);
        const bf16 *dY = m->dh[l];
        int s = run_wgrad(m, ti, g, dY, ldy, fc_input(m, l), leaf);
        if (s != PPO_OK) return join(s);
        DgradEpilogue e;
        if (l > 1) e = {m->h[l - 1], m->dh[l - 1], nullptr};
        else e = {nullptr, nullptr, d.n_lstm > 0 ? m->lstm_dtop : m->dh0_f32};
        s = run_dgrad(m, g, dY, ldy, m->shadow + m->tensors[ti].off, m->wT + m->wT_off[ti], wt_ld_of(Co), nullptr, e, st);
        if (s == PPO_OK && l > 1) s = fork_here();  // dh[l-1] is ready for the next leaf
        if (s != PPO_OK) return join(s);
    }
    if (d.n_lstm > 0) {  // through the recurrent trunk: lstm_dtop -> dh0_f32
        const int s = lstm_backward(m, rows, st);
        if (s != PPO_OK) return join(s);
    }
    if (m->ti_embed >= 0) {
        // back through the embedding: its ReLU, then weight gradient (a leaf) and input gradient (masked by the
        // ReLU of the last conv output, which the flattened vector is)
        const int te = m->ti_embed, E = d.embed;
        ConvGeom g = fc_geom(rows, m->Hs[L] * m->Ws[L] * m->Cs[L], E);
        embed_dz_kernel<<<ppo_cdiv((long long)rows * E, 256), 256, 0, st>>>(m->dh0_f32, m->h[0], m->dze, rows, E, m->hw[0]);
        PPO_LAUNCH_CHECK();
        int s = fork_here();
        if (s == PPO_OK) s = run_wgrad(m, te, g, m->dze, E, m->act[L], leaf);
        DgradEpilogue e = {m->act[L], m->dact[L], nullptr};
        if (s == PPO_OK)
            s = run_dgrad(m, g, m->dze, E, m->shadow + m->tensors[te].off, m->wT + m->wT_off[te], wt_ld_of(E), nullptr, e, st);
        if (s != PPO_OK) return join(s);
    } else {
        const int npx = m->Hs[L] * m->Ws[L], C = m->Cs[L];
        const long long total8 = (long long)rows * npx * C / 8;
        unpool_kernel<<<ppo_cdiv(total8, 256), 256, 0, st>>>(m->dh0_f32, m->act[L], m->dact[L], total8, npx, C,
                                                           m->hw[0]);
        PPO_LAUNCH_CHECK();
    }
    // With layer normalisation dact[l] arrives as the gradient of the normalised, scaled and shifted value; ln_bwd
    // turns it in place into the gradient of the convolution's output and adds the gamma and beta gradients.
    auto ln_bwd = [&](int l) -> int {
        if (!d.norm) return PPO_OK;
        const int C = m->Cs[l], tc = m->ti_conv[l];
        const long long M = (long long)rows * m->Hs[l] * m->Ws[l];
        const int lpp = C / 8;
        if (C < 16 || C > 256 || (C & (C - 1)) != 0) return PPO_ERR_UNSUPPORTED;
        int blocks = ppo_cdiv(M, (long long)8 * (32 / lpp) * 4);
        const int cap = ppo_num_sms() * 4;
        blocks = blocks > cap ? cap : (blocks < 1 ? 1 : blocks);
        if ((size_t)blocks * 2 * C > m->ln_cap) return PPO_ERR_SHAPE;
        ln_bwd_kernel<<<blocks, 256, 0, st>>>(m->dact[l], m->xhat[l], m->rstd[l], m->master + m->tensors[tc + 2].off, M, C,
                                              m->ln_part);
        PPO_LAUNCH_CHECK();
        return sum_partials(m->ln_part, blocks, C, m->grad + m->tensors[tc + 2].off, C, m->grad + m->tensors[tc + 3].off, st);
    };
    // The chain of dgrads first; then the wgrads of the GEMM layers one after the other on the caller's stream
    // with conv1's wgrad beside them on the second one.  A wgrad GEMM takes most of an SM's shared memory but
    // few registers and threads, conv1's wgrad the opposite, and both leave most issue slots and half the DRAM
    // bandwidth unused on their own, so they share the SMs.  (The dgrad kernels take whole SMs: nothing fits
    // beside them.)  Without a second stream the order is the plain one: wgrad, dgrad, layer by layer.
    for (int l = L; l >= 2; --l) {
        const int ti = m->ti_conv[l];
        ConvGeom g = conv_geom(m, l, rows);
        DgradEpilogue e = {m->act[l - 1], m->dact[l - 1], nullptr};
        e.mask_bits = m->abits[l - 1];
        int s = ln_bwd(l);
        if (s == PPO_OK && !fork)
            s = run_wgrad(m, ti, g, m->dact[l], g.Co, m->act[l - 1], st);
        if (s == PPO_OK)
            s = run_dgrad(m, g, m->dact[l], g.Co, m->shadow + m->tensors[ti].off, m->wT + m->wT_off[ti],
                          wt_ld_of(g.Co), m->wC + m->wC_off[l], e, st);
        if (s != PPO_OK) return join(s);
    }
    {
        const int s = ln_bwd(1);
        if (s != PPO_OK) return join(s);
    }
    if (fork && L >= 2) {
        int s = fork_here();  // dZ1 is ready
        if (s == PPO_OK) s = conv1_wgrad(m, mb, row0, rows, leaf);
        for (int l = 2; l <= L && s == PPO_OK; ++l) {  // conv2 first: the longest, and the best partner
            const int ti = m->ti_conv[l];
            ConvGeom g = conv_geom(m, l, rows);
            s = run_wgrad(m, ti, g, m->dact[l], g.Co, m->act[l - 1], st);
        }
        return join(s);
    }
    return join(conv1_wgrad(m, mb, row0, rows, st));
}
