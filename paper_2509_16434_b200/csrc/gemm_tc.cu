// Tensor-core versions of the encoder's implicit GEMMs for sm_100a: tcgen05.mma with the
// accumulator in tensor memory (TMEM), operands gathered into 128-byte-swizzled shared
// memory by cp.async, an mbarrier ring between the gather warps and the MMA-issuing warp,
// and a tcgen05.ld epilogue.  Every wait is bounded: on a time-out the kernel records
// PPO_ERR_TIMEOUT, drains its copies, frees its TMEM and returns.
//
//  igemm_kmajor_kernel : D[m][n] = sum_k A[m][k] B[n][k], both operands K-major.
//      forward  A = im2col(X) (row m = output pixel), B = W[co][tap][ci]
//      dgrad    A = gathered dY (row m = input pixel of one stride-parity class), B = Wt[ci][tap][co]
//  igemm_wgrad_kernel  : D[j][co] = sum_m A[m][j] B[m][co], both operands MN-major (the reduction
//      index m is the slow one in memory), split over m across CTAs, fp32 atomics into dW.
//
// Shared-memory operand image (both kernels): rows of 128 bytes (64 bf16), the 16-byte chunk c
// of row r stored at chunk position c ^ (r & 7) -- the SWIZZLE_128B pattern the UMMA shared
// memory descriptors name.  Read K-major, a row is one M/N index and its 64 columns are K; read
// MN-major, a row is one K index and its 64 columns are M/N.
#include "gemm.cuh"
#include "tcgen05.cuh"

namespace {

using namespace tc;

constexpr int kProducers = 128;       // 4 warps: gather, then epilogue
constexpr int kThreads = 160;         // wgrad kernel: + 1 warp issuing the MMAs
constexpr int kMaxTaps = 49;
// ------------------------------------------------------------------ K-major ----

constexpr int kMaxStagesK = 8;
constexpr int kGatherWarps = 8;
constexpr int kKThreads = (kGatherWarps + 5) * 32;  // gather warps, one MMA-issuing warp, 4 epilogue warps

struct Taps {
    int n;                 // taps walked along K
    signed char dy[kMaxTaps], dx[kMaxTaps];
    short wt[kMaxTaps];    // index of the tap inside the weight tensor
};

// One set of rows that share a tap list: the whole output for the forward pass, one
// stride-parity class of input pixels for dgrad.
struct KClass {
    int Hr, Wr;            // row grid: m = (b * Hr + y) * Wr + x
    long long Mrows;
    int o_oy, o_ox;        // output pixel = (y * o_mul + o_oy, x * o_mul + o_ox)
    int tile0;             // first global tile of this class
    Taps taps;
};

enum { EPI_FWD = 0, EPI_HEAD = 1, EPI_DGRAD = 2 };

struct KArgs {
    const bf16 *S;         // source [B][Hs][Ws][lds]
    int Hs, Ws, lds;
    const bf16 *Wm;        // weights: element (n, tap t, c) at n * w_row + wt[t] * w_tap + c
    int w_row, w_tap;
    int ck;                // 16-byte chunks (8 elements) per tap
    int s_mul, s_oy, s_ox; // source pixel of tap t: (y * s_mul + s_oy + dy[t], x * s_mul + s_ox + dx[t])
    int o_mul, Hout, Wout; // output row = (b * Hout + oy) * Wout + ox
    int N, BN, ldo, tiles_n;
    int stages;
    int mode, relu, A;
    const float *bias;
    bf16 *out;
    float *out_f32;
    const bf16 *mask;
    float *mean, *value;
    const float *ln_gamma, *ln_beta;  // forward with layer normalisation over the N columns of a row (null: none)
    bf16 *ln_xhat;
    float *ln_rstd;
    int32_t *status;
    int ncls, total_tiles;
    KClass cls[4];
};

struct PipeK {
    uint64_t full[kMaxStagesK];
    uint64_t empty[kMaxStagesK];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint32_t tmem_slot;
    int abort_flag;
};

// Persistent: CTA c works on tiles c, c + gridDim.x, ...  The gather warps run ahead across tile
// boundaries, the accumulator is double-buffered in TMEM so that the epilogue of one tile overlaps
// the MMAs of the next.
__global__ void __launch_bounds__(kKThreads, 1) igemm_kmajor_kernel(const __grid_constant__ KArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int BN = a.BN, S = a.stages;
    const uint32_t stage_bytes = 16384u + (uint32_t)BN * 128u;
    PipeK *pipe = reinterpret_cast<PipeK *>(smem + S * stage_bytes);
    volatile int *abort_flag = &pipe->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t acc_cols = tmem_cols_for(BN);       // columns of one accumulator
    const uint32_t ncols = acc_cols * 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe->full[s], kGatherWarps * 32);
            mbar_init(&pipe->empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&pipe->tfull[i], 1);
            mbar_init(&pipe->tempty[i], 128);
        }
        pipe->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kGatherWarps) tmem_alloc(&pipe->tmem_slot, ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = pipe->tmem_slot;
    const uint32_t smem_base = smem_u32(smem);

    if (warp < kGatherWarps) {
        // ---------------- gather: thread p owns 16-byte chunk column c = p % 8 of the K block and rows
        // p / 8 + 32 i of both tiles, so that the 8 lanes of a row read up to 128 contiguous bytes (whole
        // 32-byte sectors) and a warp writes four complete swizzled rows (no bank conflicts).
        const int p = threadIdx.x;
        const int c = p & 7, rg = p >> 3;
        const uint32_t dst0 = (uint32_t)rg * 128u + (((uint32_t)c ^ ((uint32_t)rg & 7u)) << 4);
        int it = 0;          // K blocks issued so far (all tiles)
        bool ok = true;
        for (int g = blockIdx.x; g < a.total_tiles && ok; g += gridDim.x) {
            int cl = 0;
            while (cl + 1 < a.ncls && g >= a.cls[cl + 1].tile0) ++cl;
            const KClass &k = a.cls[cl];
            const int local = g - k.tile0;
            const long long m0 = (long long)(local / a.tiles_n) * 128 + rg;
            const int n0 = (local % a.tiles_n) * BN;
            const int ntaps = k.taps.n;
            const int nkb = (ntaps * a.ck + 7) >> 3;
            // the four A rows of this thread: source pixel of tap (0, 0) and image base, or sy = INT_MIN / 2
            // for rows past the end (every tap then fails the bounds test)
            int sy[4], sx[4];
            const bf16 *img[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const long long m = m0 + 32 * i;
                if (m < k.Mrows) {
                    const int x = (int)(m % k.Wr);
                    const long long t = m / k.Wr;
                    const int y = (int)(t % k.Hr);
                    sy[i] = y * a.s_mul + a.s_oy;
                    sx[i] = x * a.s_mul + a.s_ox;
                    img[i] = a.S + (t / k.Hr) * a.Hs * a.Ws * a.lds;
                } else {
                    sy[i] = -(1 << 30);
                    sx[i] = 0;
                    img[i] = a.S;
                }
            }
            int tK = c / a.ck, cK = c % a.ck;   // tap and chunk inside the tap of flattened chunk kb * 8 + c
            const bf16 *b_src0 = a.Wm + (long long)(n0 + rg) * a.w_row;
            int nBv = (a.N - n0 - rg + 31) / 32;          // B rows of this thread that exist
            const int nBt = (BN - rg + 31) / 32;          // B rows of this thread inside the tile
            nBv = nBv < 0 ? 0 : (nBv > nBt ? nBt : nBv);
            const long long rstep = 32ll * a.w_row;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % S;
                ok = mbar_wait(&pipe->empty[s], ((it / S) & 1) ^ 1, abort_flag, a.status);
                if (!ok) break;
                const uint32_t d = smem_base + s * stage_bytes + dst0;
                const bool kv = tK < ntaps;
                const int dy = kv ? k.taps.dy[tK] : 0, dx = kv ? k.taps.dx[tK] : 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int yy = sy[i] + dy, xx = sx[i] + dx;
                    const bool v = kv && (unsigned)yy < (unsigned)a.Hs && (unsigned)xx < (unsigned)a.Ws;
                    const bf16 *src = v ? img[i] + ((yy * a.Ws + xx) * a.lds + cK * 8) : a.S;
                    cp_async16_ca(d + (uint32_t)i * 4096u, src, v);
                }
                {
                    const bf16 *src = b_src0 + (kv ? (int)k.taps.wt[tK] * a.w_tap + cK * 8 : 0);
                    const uint32_t db = d + 16384u;
                    for (int i = 0; i < nBt; ++i) {
                        const bool v = kv && i < nBv;
                        cp_async16(db + (uint32_t)i * 4096u, v ? src + i * rstep : a.Wm, v);
                    }
                }
                cK += 8;
                while (cK >= a.ck) { cK -= a.ck; ++tK; }
                cp_async_arrive(&pipe->full[s]);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
    } else if (warp == kGatherWarps) {
        // ---------------- MMA issue: one thread feeds the tensor core
        const uint32_t idesc = instr_desc(128, BN, 0, 0);
        int it = 0, ti = 0;
        bool ok = true;
        for (int g = blockIdx.x; g < a.total_tiles && ok; g += gridDim.x, ++ti) {
            int c = 0;
            while (c + 1 < a.ncls && g >= a.cls[c + 1].tile0) ++c;
            const int nkb = (a.cls[c].taps.n * a.ck + 7) >> 3;
            const int acc = ti & 1;
            ok = mbar_wait(&pipe->tempty[acc], ((ti >> 1) & 1) ^ 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t tmem_d = tmem_base + acc * acc_cols;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % S;
                ok = mbar_wait(&pipe->full[s], (it / S) & 1, abort_flag, a.status);
                if (!ok) break;
                fence_async_smem();
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t sa = smem_base + s * stage_bytes, sb = sa + 16384u;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)  // 4 x (K = 16 elements = 32 bytes along the swizzled row)
                        umma_bf16(tmem_d, smem_desc(sa + kk * 32, 16, 1024), smem_desc(sb + kk * 32, 16, 1024), idesc,
                                  (kb > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(&pipe->empty[s]);
                }
                __syncwarp();
            }
            if (ok && lane == 0) umma_commit(&pipe->tfull[acc]);
            __syncwarp();
        }
    } else {
        // ---------------- epilogue: warp w reads TMEM lanes 32 (w % 4) .. +31
        const int lg = warp & 3;
        const int p = lg * 32 + lane;
        int ti = 0;
        bool ok = true;
        for (int g = blockIdx.x; g < a.total_tiles && ok; g += gridDim.x, ++ti) {
            int c = 0;
            while (c + 1 < a.ncls && g >= a.cls[c + 1].tile0) ++c;
            const KClass &k = a.cls[c];
            const int local = g - k.tile0;
            const long long m = (long long)(local / a.tiles_n) * 128 + p;
            const int n0 = (local % a.tiles_n) * BN;
            const int nkb = (k.taps.n * a.ck + 7) >> 3;
            const bool row_ok = m < k.Mrows;
            long long orow = 0;
            if (row_ok) {
                const int x = (int)(m % k.Wr);
                const long long t = m / k.Wr;
                const int y = (int)(t % k.Hr);
                const long long b = t / k.Hr;
                orow = (b * a.Hout + (long long)y * a.o_mul + k.o_oy) * a.Wout + (long long)x * a.o_mul + k.o_ox;
            }
            const int acc = ti & 1;
            ok = mbar_wait(&pipe->tfull[acc], (ti >> 1) & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t lane_base = tmem_base + acc * acc_cols + ((uint32_t)(lg * 32) << 16);
            // Layer normalisation: the row of this thread holds all N channels of its pixel (one column tile), so it
            // walks the row twice (mean, then variance about it) before the pass that writes.
            float ln_mean = 0.f, ln_rs = 0.f;
            if (a.ln_gamma && nkb > 0) {
                float sum = 0.f;
                for (int c0 = 0; c0 < a.N; c0 += 16) {
                    float t[16];
                    tmem_ld16(lane_base + (uint32_t)c0, t);
#pragma unroll
                    for (int i = 0; i < 16; ++i) sum += t[i] + a.bias[c0 + i];
                }
                ln_mean = sum / (float)a.N;
                float sq = 0.f;
                for (int c0 = 0; c0 < a.N; c0 += 16) {
                    float t[16];
                    tmem_ld16(lane_base + (uint32_t)c0, t);
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float dlt = t[i] + a.bias[c0 + i] - ln_mean;
                        sq += dlt * dlt;
                    }
                }
                ln_rs = rsqrtf(sq / (float)a.N + kLnEps);
                if (row_ok) a.ln_rstd[orow] = ln_rs;
            }
            for (int c0 = 0; c0 < BN; c0 += 16) {
                if (n0 + c0 >= a.N) break;  // uniform across the warp
                float v[16];
                if (nkb > 0) {
                    tmem_ld16(lane_base + (uint32_t)c0, v);
                } else {  // empty reduction: the accumulator was never written
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
                if (!row_ok) continue;
                const int n = n0 + c0;
                if (a.mode == EPI_HEAD) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        if (n + i < a.A) a.mean[m * a.A + n + i] = v[i] + a.bias[n + i];
                        else if (n + i == a.A) a.value[m] = v[i] + a.bias[n + i];
                    }
                    continue;
                }
                if (a.mode == EPI_FWD) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float bv = (n + i < a.N) ? a.bias[n + i] : 0.f;
                        v[i] += bv;
                    }
                    if (a.ln_gamma) {
                        uint4 *xp = reinterpret_cast<uint4 *>(a.ln_xhat + orow * a.ldo + n);
                        uint32_t pk[8];
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = (v[i] - ln_mean) * ln_rs;
#pragma unroll
                        for (int i = 0; i < 8; ++i) pk[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
                        xp[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        xp[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fmaf(a.ln_gamma[n + i], v[i], a.ln_beta[n + i]);
                    }
                    if (a.relu) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.f);
                    }
                } else if (a.mask) {
                    const uint4 *mp = reinterpret_cast<const uint4 *>(a.mask + orow * a.ldo + n);
#pragma unroll
                    for (int hlf = 0; hlf < 2; ++hlf) {
                        if (n + hlf * 8 < a.N) {
                            const uint4 mk = mp[hlf];
                            const __nv_bfloat162 *m2 = reinterpret_cast<const __nv_bfloat162 *>(&mk);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 f = __bfloat1622float2(m2[i]);
                                if (!(f.x > 0.f)) v[hlf * 8 + 2 * i] = 0.f;
                                if (!(f.y > 0.f)) v[hlf * 8 + 2 * i + 1] = 0.f;
                            }
                        }
                    }
                }
                if (a.out) {
                    uint4 *op = reinterpret_cast<uint4 *>(a.out + orow * a.ldo + n);
#pragma unroll
                    for (int hlf = 0; hlf < 2; ++hlf) {
                        if (n + hlf * 8 < a.N) {
                            __nv_bfloat162 pk[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                pk[i] = __floats2bfloat162_rn(v[hlf * 8 + 2 * i], v[hlf * 8 + 2 * i + 1]);
                            op[hlf] = *reinterpret_cast<uint4 *>(pk);
                        }
                    }
                }
                if (a.out_f32) {
                    float4 *op = reinterpret_cast<float4 *>(a.out_f32 + orow * a.ldo + n);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (n + q * 4 < a.N) op[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                }
            }
            tc_fence_before();
            mbar_arrive(&pipe->tempty[acc]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kGatherWarps) {
        tc_fence_after();
        tmem_dealloc(tmem_base, ncols);
    }
}

// -------------------------------------------------------------------- wgrad ----

struct WArgs {
    const bf16 *X;         // [B][Hi][Wi][Ci]
    int Hi, Wi, Ci, Ho, Wo, ksz, pad;
    const bf16 *dY;        // [M][ldy]
    int ldy, Co;
    long long Mtot;        // B * Ho * Wo
    long long m_per_split; // multiple of 64
    int db64, doh64, dow64; // 64 rows = db64 images + doh64 output rows + dow64 pixels
    int Kfwd;              // ksz * ksz * Ci
    int BN;
    int stages;
    float *part;           // partial tiles [split][column tile][row tile][BN][128] fp32 (see wgrad_reduce)
    int32_t *status;
};

__global__ void __launch_bounds__(kThreads) igemm_wgrad_kernel(const __grid_constant__ WArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int BN = a.BN;
    const int nblkB = (BN + 63) >> 6;
    const uint32_t stage_bytes = 16384u + (uint32_t)nblkB * 8192u;
    const int S = a.stages;
    PipeK *pipe = reinterpret_cast<PipeK *>(smem + S * stage_bytes);
    volatile int *abort_flag = &pipe->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ncols = tmem_cols_for(BN);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe->full[s], kProducers);
            mbar_init(&pipe->empty[s], 1);
        }
        mbar_init(&pipe->tfull[0], 1);
        pipe->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(&pipe->tmem_slot, ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = pipe->tmem_slot;

    const int j0 = blockIdx.x * 128;       // tile of the (tap, ci) index
    const int co0 = blockIdx.y * BN;
    const long long m_lo = (long long)blockIdx.z * a.m_per_split;
    const long long m_hi = min(a.Mtot, m_lo + a.m_per_split);
    const int nkb = (int)((m_hi - m_lo + 63) >> 6);
    const uint32_t smem_base = smem_u32(smem);

    if (warp < 4) {
        // Thread p owns 16-byte chunk column c16 = p % 16 of the 128-column A tile (and of each pair of
        // 64-column B blocks) and rows p / 16 + 8 i, so that the lanes of a row read contiguous bytes.
        const int p = threadIdx.x;
        const int c16 = p & 15, rg = p >> 4, half = c16 >> 3, q = c16 & 7;
        int a_off = -1, a_dy = 0, a_dx = 0;   // this thread's column: offset inside a source pixel and its tap
        {
            const int jj = j0 + half * 64 + q * 8;
            if (jj < a.Kfwd) {
                const int t = jj / a.Ci;
                a_off = jj - t * a.Ci;
                a_dy = t / a.ksz - a.pad;
                a_dx = t % a.ksz - a.pad;
            }
        }
        const uint32_t dst0 = (uint32_t)half * 8192u + (uint32_t)rg * 128u + (((uint32_t)q ^ ((uint32_t)rg & 7u)) << 4);
        // output pixel of each of the 8 rows, advanced by 64 rows per K block without divisions
        int ow[8], oh[8], ob[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const long long m = m_lo + rg + 8 * i;
            ow[i] = (int)(m % a.Wo);
            const long long t = m / a.Wo;
            oh[i] = (int)(t % a.Ho);
            ob[i] = (int)(t / a.Ho);
        }
        const int co_lim = min(a.ldy, co0 + BN);  // dY columns that exist in memory for this tile
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % S;
            ok = mbar_wait(&pipe->empty[s], ((kb / S) & 1) ^ 1, abort_flag, a.status);
            if (!ok) break;
            const uint32_t sa = smem_base + s * stage_bytes + dst0, sb = sa + 16384u - (uint32_t)half * 8192u;
            const long long mb = m_lo + (long long)kb * 64 + rg;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const long long m = mb + 8 * i;
                const bool row_ok = m < m_hi;
                const int yy = 2 * oh[i] + a_dy, xx = 2 * ow[i] + a_dx;
                const bool v = row_ok && a_off >= 0 && (unsigned)yy < (unsigned)a.Hi && (unsigned)xx < (unsigned)a.Wi;
                const bf16 *src = v ? a.X + (((long long)ob[i] * a.Hi + yy) * a.Wi + xx) * a.Ci + a_off : a.X;
                cp_async16_ca(sa + (uint32_t)i * 1024u, src, v);
                const bf16 *dyrow = a.dY + m * a.ldy;
                for (int blk = half; blk < nblkB; blk += 2) {
                    const int co = co0 + blk * 64 + q * 8;
                    const bool vb = row_ok && co < co_lim;
                    cp_async16(sb + (uint32_t)blk * 8192u + (uint32_t)i * 1024u, vb ? dyrow + co : a.dY, vb);
                }
                // next K block: 64 rows further
                ow[i] += a.dow64;
                if (ow[i] >= a.Wo) { ow[i] -= a.Wo; ++oh[i]; }
                oh[i] += a.doh64;
                if (oh[i] >= a.Ho) { oh[i] -= a.Ho; ++ob[i]; }
                ob[i] += a.db64;
            }
            cp_async_arrive(&pipe->full[s]);
        }
        cp_async_commit();
        cp_async_wait<0>();

        // ---------------- epilogue: TMEM lane p is column j0 + p of dW^T
        if (ok && nkb > 0) ok = mbar_wait(&pipe->tfull[0], 0, abort_flag, a.status);
        tc_fence_after();
        if (ok && nkb > 0) {
            float *tile = a.part + ((size_t)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * (size_t)(128 * BN);
            const uint32_t lane_base = tmem_d + ((uint32_t)(warp * 32) << 16);
            for (int c0 = 0; c0 < BN; c0 += 16) {
                float v[16];
                tmem_ld16(lane_base + (uint32_t)c0, v);
#pragma unroll
                for (int i = 0; i < 16; ++i) tile[(c0 + i) * 128 + p] = v[i];
            }
        }
    } else {
        const uint32_t idesc = instr_desc(128, BN, 1, 1);
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % S;
            ok = mbar_wait(&pipe->full[s], (kb / S) & 1, abort_flag, a.status);
            if (!ok) break;
            fence_async_smem();
            tc_fence_after();
            if (lane == 0) {
                const uint32_t sa = smem_base + s * stage_bytes, sb = sa + 16384u;
#pragma unroll
                for (int k = 0; k < 4; ++k)  // 4 x (K = 16 reduction rows = 2048 bytes)
                    umma_bf16(tmem_d, smem_desc(sa + k * 2048, 8192, 1024), smem_desc(sb + k * 2048, 8192, 1024),
                              idesc, (kb > 0 || k > 0) ? 1u : 0u);
                umma_commit(&pipe->empty[s]);
            }
            __syncwarp();
        }
        if (ok && nkb > 0 && lane == 0) umma_commit(&pipe->tfull[0]);
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem_d, ncols);
    }
}

// --------------------------------------------------------------------- host ----

int pick_bn(int N) {  // tile width: N split evenly into tiles of at most 256, rounded up to 16
    const int tiles = (N + 255) / 256;
    int bn = ((N + tiles - 1) / tiles + 15) / 16 * 16;
    return bn < 16 ? 16 : bn;
}

int kmajor_stages(int BN) {
    int s = (int)((200 * 1024) / (16384 + (size_t)BN * 128));
    return s > kMaxStagesK ? kMaxStagesK : (s < 3 ? 3 : s);
}
size_t kmajor_smem(int BN) { return (size_t)kmajor_stages(BN) * (16384 + (size_t)BN * 128) + sizeof(PipeK) + 1024; }
int wgrad_stages(int BN) {
    int s = (int)((200 * 1024) / (16384 + (size_t)((BN + 63) / 64) * 8192));
    return s > kMaxStagesK ? kMaxStagesK : (s < 3 ? 3 : s);
}
size_t wgrad_smem(int BN) {
    return (size_t)wgrad_stages(BN) * (16384 + (size_t)((BN + 63) / 64) * 8192) + sizeof(PipeK) + 1024;
}

// Opts both kernels into their largest dynamic shared memory footprint, once per device.
int ensure_smem_attrs() {
    static bool attr_set[64] = {false};
    int dev = 0;
    PPO_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return PPO_ERR_CUDA;
    if (!attr_set[dev]) {
        size_t mx = 0;
        for (int bn = 16; bn <= 256; bn += 16) mx = kmajor_smem(bn) > mx ? kmajor_smem(bn) : mx;
        PPO_CUDA_CHECK(cudaFuncSetAttribute(igemm_kmajor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mx));
        size_t mw = 0;
        for (int bn = 16; bn <= 256; bn += 16) mw = wgrad_smem(bn) > mw ? wgrad_smem(bn) : mw;
        PPO_CUDA_CHECK(cudaFuncSetAttribute(igemm_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mw));
        attr_set[dev] = true;
    }
    return PPO_OK;
}

// Fills the tile bookkeeping of a.cls[0 .. ncls) (Mrows, taps set by the caller) and launches.
int launch_kmajor(KArgs &a, cudaStream_t st) {
    int s = ensure_smem_attrs();
    if (s != PPO_OK) return s;
    a.tiles_n = (a.N + a.BN - 1) / a.BN;
    long long tiles = 0;
    for (int c = 0; c < a.ncls; ++c) {
        a.cls[c].tile0 = (int)tiles;
        tiles += ((a.cls[c].Mrows + 127) / 128) * a.tiles_n;
    }
    if (tiles <= 0) return PPO_OK;
    if (tiles > 0x7fffffffll) return PPO_ERR_UNSUPPORTED;
    a.total_tiles = (int)tiles;
    a.stages = kmajor_stages(a.BN);
    const int sms = ppo_num_sms();
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    igemm_kmajor_kernel<<<grid, kKThreads, kmajor_smem(a.BN), st>>>(a);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

}  // namespace

int tc_gemm_fwd(const ConvGeom &g, const bf16 *X, const bf16 *W, const FwdEpilogue &e, int32_t *status,
                cudaStream_t st) {
    if (g.Ci % 8 != 0 || g.taps() > kMaxTaps || !status) return PPO_ERR_UNSUPPORTED;
    KArgs a = {};
    a.S = X; a.Hs = g.Hi; a.Ws = g.Wi; a.lds = g.Ci;
    a.Wm = W; a.w_row = g.K(); a.w_tap = g.Ci; a.ck = g.Ci / 8;
    a.s_mul = 2; a.s_oy = a.s_ox = -g.pad;
    a.o_mul = 1; a.Hout = g.Ho; a.Wout = g.Wo;
    a.N = g.Co; a.BN = pick_bn(g.Co); a.ldo = e.ldo ? e.ldo : g.Co;
    a.mode = e.out ? EPI_FWD : EPI_HEAD; a.relu = e.relu; a.A = e.A;
    if (e.ln_gamma) {
        if (!e.ln_beta || !e.ln_xhat || !e.ln_rstd || !e.out || g.Co > 256 || g.Co % 16 != 0 || a.ldo != g.Co) return PPO_ERR_UNSUPPORTED;
        a.ln_gamma = e.ln_gamma; a.ln_beta = e.ln_beta; a.ln_xhat = e.ln_xhat; a.ln_rstd = e.ln_rstd;
    }
    a.bias = e.bias; a.out = e.out; a.out_f32 = nullptr; a.mask = nullptr; a.mean = e.out_mean; a.value = e.out_value;
    a.status = status;
    a.ncls = 1;
    KClass &k = a.cls[0];
    k.Hr = g.Ho; k.Wr = g.Wo; k.Mrows = g.M(); k.o_oy = k.o_ox = 0;
    k.taps.n = g.taps();
    for (int t = 0; t < g.taps(); ++t) {
        k.taps.dy[t] = (signed char)(t / g.k);
        k.taps.dx[t] = (signed char)(t % g.k);
        k.taps.wt[t] = (short)t;
    }
    if (a.mode == EPI_FWD && g.Co % 8 != 0) return PPO_ERR_UNSUPPORTED;
    return launch_kmajor(a, st);
}

int tc_gemm_dgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *Wt, int wt_ld, const DgradEpilogue &e,
                  int32_t *status, cudaStream_t st) {
    if (g.Ci % 8 != 0 || ldy % 8 != 0 || wt_ld % 8 != 0 || ldy < wt_ld || !status) return PPO_ERR_UNSUPPORTED;
    KArgs a = {};
    a.S = dY; a.Hs = g.Ho; a.Ws = g.Wo; a.lds = ldy;
    a.Wm = Wt; a.w_row = g.taps() * wt_ld; a.w_tap = wt_ld; a.ck = wt_ld / 8;
    a.s_mul = 1; a.s_oy = a.s_ox = 0;
    a.o_mul = 2; a.Hout = g.Hi; a.Wout = g.Wi;
    a.N = g.Ci; a.BN = pick_bn(g.Ci); a.ldo = g.Ci;
    a.mode = EPI_DGRAD; a.relu = 0; a.A = 0;
    a.bias = nullptr; a.out = e.out; a.out_f32 = e.out_f32; a.mask = e.mask_act;
    a.status = status;
    // One class per stride parity (ih % 2, iw % 2): inside a class every input pixel sees the same
    // kernel taps, kh = (ph + pad) mod 2, +2, ..., each reading output row (ih + pad - kh) / 2.
    // A class no tap reaches (k = 1, odd pixels) still runs so that its outputs are written as zeros.
    a.ncls = 0;
    for (int ph = 0; ph < 2; ++ph)
        for (int pw = 0; pw < 2; ++pw) {
            const int Hr = (g.Hi - ph + 1) / 2, Wr = (g.Wi - pw + 1) / 2;
            if (Hr <= 0 || Wr <= 0) continue;
            KClass &k = a.cls[a.ncls++];
            k.Hr = Hr; k.Wr = Wr; k.Mrows = (long long)g.B * Hr * Wr;
            k.o_oy = ph; k.o_ox = pw;
            int nt = 0;
            for (int kh = (ph + g.pad) & 1; kh < g.k; kh += 2)
                for (int kw = (pw + g.pad) & 1; kw < g.k; kw += 2) {
                    if (nt >= kMaxTaps) return PPO_ERR_UNSUPPORTED;
                    k.taps.dy[nt] = (signed char)((ph + g.pad - kh) / 2);
                    k.taps.dx[nt] = (signed char)((pw + g.pad - kw) / 2);
                    k.taps.wt[nt] = (short)(kh * g.k + kw);
                    ++nt;
                }
            k.taps.n = nt;
        }
    return launch_kmajor(a, st);
}

int tc_gemm_wgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW, float *part, size_t part_elems,
                  int32_t *status, cudaStream_t st) {
    if (g.Ci % 8 != 0 || ldy % 8 != 0 || !status || !part) return PPO_ERR_UNSUPPORTED;
    WArgs a = {};
    a.X = X; a.Hi = g.Hi; a.Wi = g.Wi; a.Ci = g.Ci; a.Ho = g.Ho; a.Wo = g.Wo; a.ksz = g.k; a.pad = g.pad;
    a.dY = dY; a.ldy = ldy; a.Co = g.Co;
    a.Mtot = g.M();
    a.Kfwd = g.K();
    a.BN = pick_bn(g.Co);
    a.stages = wgrad_stages(a.BN);
    a.part = part;
    a.status = status;
    int s = ensure_smem_attrs();
    if (s != PPO_OK) return s;
    const int jtiles = (a.Kfwd + 127) / 128, ctiles = (g.Co + a.BN - 1) / a.BN;
    const int tiles = jtiles * ctiles;
    long long splits = (long long)ppo_num_sms() * 2 / tiles;
    if (splits < 1) splits = 1;
    const size_t per_split = (size_t)tiles * 128 * a.BN;
    if ((size_t)splits * per_split > part_elems) splits = (long long)(part_elems / per_split);  // the scratch bounds the split
    if (splits < 1) return PPO_ERR_SHAPE;
    long long per = ((a.Mtot + splits - 1) / splits + 63) / 64 * 64;
    if (per < 256) per = 256;
    splits = (a.Mtot + per - 1) / per;
    a.m_per_split = per;
    a.db64 = 64 / (g.Ho * g.Wo);
    a.doh64 = (64 % (g.Ho * g.Wo)) / g.Wo;
    a.dow64 = 64 % g.Wo;
    dim3 grid((unsigned)((a.Kfwd + 127) / 128), (unsigned)((g.Co + a.BN - 1) / a.BN), (unsigned)splits);
    igemm_wgrad_kernel<<<grid, kThreads, wgrad_smem(a.BN), st>>>(a);
    PPO_LAUNCH_CHECK();
    return wgrad_reduce(part, jtiles, ctiles, (int)splits, a.BN, a.Kfwd, g.Co, dW, nullptr, 0, st);
}
