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

namespace {

constexpr int kProducers = 128;       // 4 warps: gather, then epilogue
constexpr int kThreads = 160;         // wgrad kernel: + 1 warp issuing the MMAs
constexpr int kMaxTaps = 49;
constexpr long long kWaitCycles = 4000000000ll;  // ~2 s at 2 GHz

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; returns false when this or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int32_t *status) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            ppo_report(status, PPO_ERR_TIMEOUT);
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
    const uint32_t n = valid ? 16u : 0u;  // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// The mbarrier receives one arrival from this thread once all cp.async it has issued so far have
// landed (the arrival counts against the barrier's expected count).
__device__ __forceinline__ void cp_async_arrive(uint64_t *bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Orders generic-proxy writes to shared memory that this thread has observed (here: the gather
// warps' cp.async data, observed through the full barrier) before its later async-proxy
// operations (the tensor core reads operands through the async proxy).
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t *slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], bf16 operands, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
        "%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor for the SWIZZLE_128B image: start address, leading and
// stride byte offsets (each >> 4), descriptor version 1 (bit 46), layout type 2 (bits 61-63).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1),
// operand majors (bit 15, 16: 0 = K-major, 1 = MN-major), N >> 3 (bits 17-22), M >> 4 (bits 24-28).
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ uint32_t tmem_cols_for(int bn) {
    uint32_t c = 32;
    while ((int)c < bn) c <<= 1;
    return c;
}

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
        // ---------------- gather: thread p fills half h = p / 128 (4 of the 8 chunks) of row p % 128 of the
        // A tile, and chunk slot p % 8 of B rows p/8, p/8 + 32, ...
        const int p = threadIdx.x;
        const int r = p & 127, h = p >> 7;
        const int jB = p & 7, rB = p >> 3;
        const uint32_t sw = (uint32_t)(r & 7);
        const uint32_t a_dst0 = (uint32_t)r * 128u;
        const uint32_t b_dst0 = 16384u + (uint32_t)rB * 128u + (((uint32_t)jB ^ ((uint32_t)rB & 7u)) << 4);
        const bool fast = (a.ck & 3) == 0;   // a group of 4 chunks never straddles two taps
        int it = 0;          // K blocks issued so far (all tiles)
        bool ok = true;
        for (int g = blockIdx.x; g < a.total_tiles && ok; g += gridDim.x) {
            int c = 0;
            while (c + 1 < a.ncls && g >= a.cls[c + 1].tile0) ++c;
            const KClass &k = a.cls[c];
            const int local = g - k.tile0;
            const long long m = (long long)(local / a.tiles_n) * 128 + r;
            const int n0 = (local % a.tiles_n) * BN;
            const int ntaps = k.taps.n;
            const int nkb = (ntaps * a.ck + 7) >> 3;
            const bool row_ok = m < k.Mrows;
            int y = 0, x = 0;
            long long b = 0;
            if (row_ok) {
                x = (int)(m % k.Wr);
                const long long t = m / k.Wr;
                y = (int)(t % k.Hr);
                b = t / k.Hr;
            }
            const int sy0 = y * a.s_mul + a.s_oy, sx0 = x * a.s_mul + a.s_ox;
            const bf16 *src_img = a.S + b * a.Hs * a.Ws * a.lds;
            // A walk: flattened chunk index of this thread's group is kb * 8 + 4 h
            int tA = (4 * h) / a.ck, cA = (4 * h) % a.ck;
            // B walk: flattened chunk index kb * 8 + jB
            int tB = jB / a.ck, cB = jB % a.ck;
            const bf16 *b_src0 = a.Wm + (long long)(n0 + rB) * a.w_row;
            int nBv = (a.N - n0 - rB + 31) / 32;          // B rows of this thread that exist
            const int nBt = (BN - rB + 31) / 32;          // B rows of this thread inside the tile
            nBv = nBv < 0 ? 0 : (nBv > nBt ? nBt : nBv);
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % S;
                ok = mbar_wait(&pipe->empty[s], ((it / S) & 1) ^ 1, abort_flag, a.status);
                if (!ok) break;
                const uint32_t st = smem_base + s * stage_bytes;
                if (fast) {
                    bool v = row_ok && tA < ntaps;
                    const bf16 *src = a.S;
                    if (v) {
                        const int yy = sy0 + k.taps.dy[tA], xx = sx0 + k.taps.dx[tA];
                        v = (unsigned)yy < (unsigned)a.Hs && (unsigned)xx < (unsigned)a.Ws;
                        if (v) src = src_img + ((yy * a.Ws + xx) * a.lds + cA * 8);
                    }
                    const uint32_t d = st + a_dst0;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        cp_async16(d + ((((uint32_t)(4 * h + j)) ^ sw) << 4), src + j * 8, v);
                    cA += 8;
                    while (cA >= a.ck) { cA -= a.ck; ++tA; }
                } else {
                    int t = tA, cc = cA;
                    for (int j = 0; j < 4; ++j) {
                        while (cc >= a.ck) { cc -= a.ck; ++t; }
                        bool v = row_ok && t < ntaps;
                        const bf16 *src = a.S;
                        if (v) {
                            const int yy = sy0 + k.taps.dy[t], xx = sx0 + k.taps.dx[t];
                            v = (unsigned)yy < (unsigned)a.Hs && (unsigned)xx < (unsigned)a.Ws;
                            if (v) src = src_img + ((yy * a.Ws + xx) * a.lds + cc * 8);
                        }
                        cp_async16(st + a_dst0 + ((((uint32_t)(4 * h + j)) ^ sw) << 4), src, v);
                        ++cc;
                    }
                    cA += 8;
                    while (cA >= a.ck) { cA -= a.ck; ++tA; }
                }
                {
                    const bool kv = tB < ntaps;
                    const bf16 *src = b_src0 + (kv ? (int)k.taps.wt[tB] * a.w_tap + cB * 8 : 0);
                    const uint32_t d = st + b_dst0;
                    const long long rstep = 32ll * a.w_row;
                    for (int i = 0; i < nBt; ++i) {
                        const bool v = kv && i < nBv;
                        cp_async16(d + (uint32_t)i * 4096u, v ? src + i * rstep : a.Wm, v);
                    }
                    cB += 8;
                    while (cB >= a.ck) { cB -= a.ck; ++tB; }
                }
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
                        if (a.relu) v[i] = fmaxf(v[i], 0.f);
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
    int Kfwd;              // ksz * ksz * Ci
    int BN;
    int stages;
    float *dW;             // [Co][Kfwd], accumulated with atomics
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
        const int p = threadIdx.x;
        const int r = p & 63, half = p >> 6;
        // this thread's 8 A chunks: columns j0 + half*64 + 8 q, fixed for the whole kernel
        int a_off[8];       // element offset of the chunk inside a source pixel, or -1 when past Kfwd
        signed char a_dy[8], a_dx[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int jj = j0 + half * 64 + q * 8;
            if (jj < a.Kfwd) {
                const int t = jj / a.Ci;
                a_off[q] = jj - t * a.Ci;
                a_dy[q] = (signed char)(t / a.ksz);
                a_dx[q] = (signed char)(t % a.ksz);
            } else {
                a_off[q] = -1;
                a_dy[q] = a_dx[q] = 0;
            }
        }
        const int co_lim = min(a.ldy, co0 + BN);  // dY columns that exist in memory for this tile
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % S;
            ok = mbar_wait(&pipe->empty[s], ((kb / S) & 1) ^ 1, abort_flag, a.status);
            if (!ok) break;
            const uint32_t sa = smem_base + s * stage_bytes, sb = sa + 16384u;
            const long long m = m_lo + (long long)kb * 64 + r;
            const bool row_ok = m < m_hi;
            int oh = 0, ow = 0;
            long long b = 0;
            if (row_ok) {
                ow = (int)(m % a.Wo);
                const long long t = m / a.Wo;
                oh = (int)(t % a.Ho);
                b = t / a.Ho;
            }
            const int y0 = 2 * oh - a.pad, x0 = 2 * ow - a.pad;
            const bf16 *img = a.X + b * a.Hi * a.Wi * a.Ci;
            const uint32_t arow = sa + half * 8192 + r * 128;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int yy = y0 + a_dy[q], xx = x0 + a_dx[q];
                const bool v = row_ok && a_off[q] >= 0 && yy >= 0 && yy < a.Hi && xx >= 0 && xx < a.Wi;
                const bf16 *src = v ? img + ((long long)yy * a.Wi + xx) * a.Ci + a_off[q] : a.X;
                cp_async16(arow + ((q ^ (r & 7)) << 4), src, v);
            }
            const bf16 *dyrow = a.dY + m * a.ldy;
            for (int blk = half; blk < nblkB; blk += 2) {
                const uint32_t brow = sb + blk * 8192 + r * 128;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int co = co0 + blk * 64 + q * 8;
                    const bool v = row_ok && co < co_lim;
                    cp_async16(brow + ((q ^ (r & 7)) << 4), v ? dyrow + co : a.dY, v);
                }
            }
            cp_async_arrive(&pipe->full[s]);
        }
        cp_async_commit();
        cp_async_wait<0>();

        // ---------------- epilogue: TMEM lane p is column j0 + p of dW^T
        if (ok && nkb > 0) ok = mbar_wait(&pipe->tfull[0], 0, abort_flag, a.status);
        tc_fence_after();
        if (ok && nkb > 0) {
            const int jj = j0 + p;
            const uint32_t lane_base = tmem_d + ((uint32_t)(warp * 32) << 16);
            for (int c0 = 0; c0 < BN; c0 += 16) {
                if (co0 + c0 >= a.Co) break;
                float v[16];
                tmem_ld16(lane_base + (uint32_t)c0, v);
                if (jj >= a.Kfwd) continue;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int co = co0 + c0 + i;
                    if (co < a.Co) atomicAdd(a.dW + (long long)co * a.Kfwd + jj, v[i]);
                }
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
    a.N = g.Co; a.BN = pick_bn(g.Co); a.ldo = g.Co;
    a.mode = e.out ? EPI_FWD : EPI_HEAD; a.relu = e.relu; a.A = e.A;
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

int tc_gemm_wgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW, int32_t *status,
                  cudaStream_t st) {
    if (g.Ci % 8 != 0 || ldy % 8 != 0 || !status) return PPO_ERR_UNSUPPORTED;
    WArgs a = {};
    a.X = X; a.Hi = g.Hi; a.Wi = g.Wi; a.Ci = g.Ci; a.Ho = g.Ho; a.Wo = g.Wo; a.ksz = g.k; a.pad = g.pad;
    a.dY = dY; a.ldy = ldy; a.Co = g.Co;
    a.Mtot = g.M();
    a.Kfwd = g.K();
    a.BN = pick_bn(g.Co);
    a.stages = wgrad_stages(a.BN);
    a.dW = dW;
    a.status = status;
    int s = ensure_smem_attrs();
    if (s != PPO_OK) return s;
    const int tiles = ((a.Kfwd + 127) / 128) * ((g.Co + a.BN - 1) / a.BN);
    long long splits = (long long)ppo_num_sms() * 2 / tiles;
    if (splits < 1) splits = 1;
    long long per = ((a.Mtot + splits - 1) / splits + 63) / 64 * 64;
    if (per < 256) per = 256;
    splits = (a.Mtot + per - 1) / per;
    a.m_per_split = per;
    dim3 grid((unsigned)((a.Kfwd + 127) / 128), (unsigned)((g.Co + a.BN - 1) / a.BN), (unsigned)splits);
    igemm_wgrad_kernel<<<grid, kThreads, wgrad_smem(a.BN), st>>>(a);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}
