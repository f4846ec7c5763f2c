// First convolution (one input channel) on the tensor cores.
//
// Per output pixel the layer is a dot product of k*k depth values with each of C1 filters: far too short a
// reduction for the CUDA cores to do cheaply (C1 * k*k multiply-adds per pixel, one instruction each), but
// one tcgen05.mma of K = 16 covers a 3x3 window for 128 pixels and all filters at once.  Producer threads
// build the im2col tile themselves -- one pixel per thread, its k*k fp16 depth values (zero padded to a
// multiple of 16) -- directly in the unswizzled K-major core-matrix layout (8 rows x 16 bytes per core
// matrix); the filters are converted from the bf16 shadow to fp16 once per CTA, so that both operands are
// fp16 and the depth values enter exactly.  fp32 accumulation in tensor memory, bias + ReLU + bf16 in the
// epilogue, which also writes the one-bit ReLU gates the backward pass reads.
#include "gemm.cuh"
#include "tcgen05.cuh"

namespace {

using namespace tc;

constexpr int kMaxStages = 8;
constexpr int kProdGroups = 4;  // groups of 128 producer threads; group g builds sub-tile g of every stage
constexpr int kEpiWarps = 8;    // two per TMEM lane quarter, alternate 16-column chunks
constexpr int kThreads = (kProdGroups * 4 + 1 + kEpiWarps) * 32;

struct Args {
    const __half *depth;
    const bf16 *W;      // [C1][k*k] bf16
    const float *bias;  // [C1]
    bf16 *out;          // [M][C1]
    uint32_t *bits;     // [M][C1 / 32] or null
    long long M;        // output pixels
    int Hi, Wi, Ho, Wo, C1, KP;  // KP = k*k rounded up to 16
    int tiles;   // 128-pixel tiles
    int T;       // tiles per stage (one barrier round trip and one accumulator hand-over per T tiles)
    int stages;
    int32_t *status;
};

struct Pipe {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tfull[4];
    uint64_t tempty[4];
    uint32_t tmem_slot;
    int abort_flag;
    alignas(16) float bias[256];
};

// Unswizzled K-major operand image: element (row r, column k) of a tile with KP columns lives at
// (r / 8) * (KP / 8) * 128 + (k / 8) * 128 + (r % 8) * 16 + (k % 8) * 2 bytes.
__device__ __forceinline__ uint32_t core_offset(int r, int kchunk, int KP) {
    return (uint32_t)(r >> 3) * (uint32_t)(KP >> 3) * 128u + (uint32_t)kchunk * 128u + (uint32_t)(r & 7) * 16u;
}

__device__ __forceinline__ uint64_t desc_nosw(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

// kind::f16 with fp16 A and B (format 0), fp32 D, both K-major.
__host__ __device__ constexpr uint32_t idesc_f16(int M, int N) {
    return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

template <int KS>
__global__ void __launch_bounds__(kThreads, 1) conv1_tc_kernel(const __grid_constant__ Args a) {
    constexpr int K2 = KS * KS, KP = (K2 + 15) / 16 * 16, P = KS / 2;
    constexpr uint32_t kTileBytes = 128u * KP * 2u;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int N = a.C1, T = a.T, S = a.stages;
    const uint32_t stage_bytes = (uint32_t)T * kTileBytes;
    uint8_t *bsm = smem + (size_t)S * stage_bytes;                 // filters [N][KP] fp16
    Pipe *pipe = reinterpret_cast<Pipe *>(bsm + ((N * KP * 2 + 1023) / 1024) * 1024);
    volatile int *abort_flag = &pipe->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t acc_cols = tmem_cols_for(T * N);                // T accumulators side by side
    const int nacc_log = acc_cols * 4 <= 512 ? 2 : 1, nacc = 1 << nacc_log;
    const uint32_t ncols = acc_cols * nacc;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe->full[s], T * 128);
            mbar_init(&pipe->empty[s], 1);
        }
        for (int i = 0; i < nacc; ++i) {
            mbar_init(&pipe->tfull[i], 1);
            mbar_init(&pipe->tempty[i], kEpiWarps * 32);
        }
        pipe->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = threadIdx.x; i < N; i += kThreads) pipe->bias[i] = a.bias[i];
    // filters: zero padded columns included
    for (int i = threadIdx.x; i < N * KP; i += kThreads) {
        const int n = i / KP, k = i - n * KP;
        const __half h = k < K2 ? __float2half_rn(bf2f(a.W[n * K2 + k])) : __float2half_rn(0.f);
        *reinterpret_cast<__half *>(bsm + core_offset(n, k >> 3, KP) + (k & 7) * 2) = h;
    }
    fence_async_smem();
    if (warp == kProdGroups * 4) tmem_alloc(&pipe->tmem_slot, ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = pipe->tmem_slot;
    const uint32_t smem_base = smem_u32(smem);

    // contiguous run of stages (T tiles each) for this CTA
    const int nstage_all = (a.tiles + T - 1) / T;
    const int q = nstage_all / (int)gridDim.x, rem = nstage_all - q * (int)gridDim.x, b = (int)blockIdx.x;
    const int s0 = b * q + (b < rem ? b : rem), ns = q + (b < rem ? 1 : 0);

    if (warp < kProdGroups * 4) {
        // ---------------- producers: one output pixel per thread and stage
        const int grp = warp >> 2, r = threadIdx.x & 127;
        if (grp < T) {
            bool ok = true;
            // output pixel of this thread in its first stage, then advanced by T * 128 pixels per stage without
            // divisions
            const int step = T * 128, hw = a.Ho * a.Wo;
            const int d_b = step / hw, d_oh = (step % hw) / a.Wo, d_ow = step % a.Wo;
            int ow, oh, ib;
            long long m = ((long long)s0 * T + grp) * 128 + r;
            {
                ow = (int)(m % a.Wo);
                const long long t = m / a.Wo;
                oh = (int)(t % a.Ho);
                ib = (int)(t / a.Ho);
            }
            int s = 0;
            uint32_t ph = 0;
            for (int li = 0; li < ns && ok; ++li, m += step) {
                ok = mbar_wait(&pipe->empty[s], ph ^ 1u, abort_flag, a.status);
                if (!ok) break;
                unsigned short hv[KP];
#pragma unroll
                for (int k = 0; k < KP; ++k) hv[k] = 0;
                if (m < a.M) {
                    const unsigned short *img =
                        reinterpret_cast<const unsigned short *>(a.depth) + (long long)ib * a.Hi * a.Wi;
#pragma unroll
                    for (int kh = 0; kh < KS; ++kh) {
                        const int ih = 2 * oh + kh - P;
#pragma unroll
                        for (int kw = 0; kw < KS; ++kw) {
                            const int iw = 2 * ow + kw - P;
                            if (ih >= 0 && ih < a.Hi && iw >= 0 && iw < a.Wi) hv[kh * KS + kw] = __ldg(img + ih * a.Wi + iw);
                        }
                    }
                }
                uint8_t *dst = smem + (size_t)s * stage_bytes + (size_t)grp * kTileBytes;
#pragma unroll
                for (int c = 0; c < KP / 8; ++c) {
                    uint4 v;
                    v.x = hv[8 * c] | ((uint32_t)hv[8 * c + 1] << 16);
                    v.y = hv[8 * c + 2] | ((uint32_t)hv[8 * c + 3] << 16);
                    v.z = hv[8 * c + 4] | ((uint32_t)hv[8 * c + 5] << 16);
                    v.w = hv[8 * c + 6] | ((uint32_t)hv[8 * c + 7] << 16);
                    *reinterpret_cast<uint4 *>(dst + core_offset(r, c, KP)) = v;
                }
                fence_async_smem();
                mbar_arrive(&pipe->full[s]);
                ow += d_ow;
                if (ow >= a.Wo) { ow -= a.Wo; ++oh; }
                oh += d_oh;
                if (oh >= a.Ho) { oh -= a.Ho; ++ib; }
                ib += d_b;
                if (++s == S) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == kProdGroups * 4) {
        // ---------------- MMA issue: T tiles per stage, each into its own columns of the accumulator
        const uint32_t idesc = idesc_f16(128, N);
        const uint32_t sbo = (uint32_t)(KP >> 3) * 128u;
        const uint64_t dB = desc_nosw(smem_u32(bsm), 128u, sbo);
        const uint64_t dA0 = desc_nosw(smem_base, 128u, sbo);
        const uint32_t a_hi = (uint32_t)(dA0 >> 32), b_hi = (uint32_t)(dB >> 32);
        bool ok = true;
        int s = 0;
        uint32_t ph = 0;
        for (int li = 0; li < ns && ok; ++li) {
            const int acc = li & (nacc - 1);
            ok = mbar_wait(&pipe->tempty[acc], ((li >> nacc_log) & 1) ^ 1, abort_flag, a.status);
            if (!ok) break;
            ok = mbar_wait(&pipe->full[s], ph, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                uint32_t la = (uint32_t)dA0 + (uint32_t)s * (stage_bytes >> 4);
                uint32_t td = tmem_base + acc * acc_cols;
                for (int g = 0; g < T; ++g, la += kTileBytes >> 4, td += N) {
#pragma unroll
                    for (int kk = 0; kk < KP / 16; ++kk)  // 16 columns = two core matrices = 256 bytes
                        umma_bf16_lh(td, la + kk * 16, a_hi, (uint32_t)dB + kk * 16, b_hi, idesc, kk > 0 ? 1u : 0u);
                }
                umma_commit(&pipe->empty[s]);
                umma_commit(&pipe->tfull[acc]);
            }
            __syncwarp();
            if (++s == S) { s = 0; ph ^= 1u; }
        }
    } else {
        // ---------------- epilogue: TMEM lane = pixel of a tile; warp w reads lanes 32 (w % 4) .. +31
        const int lg = warp & 3, half = (warp - (kProdGroups * 4 + 1)) >> 2;
        const int p = lg * 32 + lane;
        unsigned short *bits16 = reinterpret_cast<unsigned short *>(a.bits);
        float bv[16];  // with N = 32 a warp always meets the same 16 columns
#pragma unroll
        for (int i = 0; i < 16; ++i) bv[i] = pipe->bias[(half * 16 + i) % N];
        const bool fixed_cols = N == 32;
        bool ok = true;
        for (int li = 0; li < ns && ok; ++li) {
            const int acc = li & (nacc - 1);
            ok = mbar_wait(&pipe->tfull[acc], (li >> nacc_log) & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t lane_base = tmem_base + acc * acc_cols + ((uint32_t)(lg * 32) << 16);
            for (int cc = half * 16; cc < T * N; cc += 32) {   // column of the accumulator: tile g, channel c0
                const int g = cc / N, c0 = cc - g * N;
                const long long m = ((long long)(s0 + li) * T + g) * 128 + p;
                float v[16];
                tmem_ld16(lane_base + (uint32_t)cc, v);
                uint4 o[2];
                __nv_bfloat162 *pk = reinterpret_cast<__nv_bfloat162 *>(o);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float b0 = fixed_cols ? bv[2 * j] : pipe->bias[c0 + 2 * j];
                    const float b1 = fixed_cols ? bv[2 * j + 1] : pipe->bias[c0 + 2 * j + 1];
                    v[2 * j] = fmaxf(v[2 * j] + b0, 0.f);
                    v[2 * j + 1] = fmaxf(v[2 * j + 1] + b1, 0.f);
                    pk[j] = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
                }
                if (m < a.M) {
                    uint4 *op = reinterpret_cast<uint4 *>(a.out + m * N + c0);
                    op[0] = o[0];
                    op[1] = o[1];
                    if (bits16) {  // 16 gate bits = one half of a 32-channel word
                        uint32_t gate = 0;
#pragma unroll
                        for (int i = 0; i < 16; ++i) gate |= (v[i] > 0.f ? 1u : 0u) << i;
                        bits16[m * (N >> 4) + (c0 >> 4)] = (unsigned short)gate;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&pipe->tempty[acc]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProdGroups * 4) {
        tc_fence_after();
        tmem_dealloc(tmem_base, ncols);
    }
}

template <int KS>
int launch(Args &a, cudaStream_t st) {
    constexpr int KP = (KS * KS + 15) / 16 * 16;
    // tiles per stage: as many accumulators as fit twice into the 512 columns of tensor memory, at most one per
    // producer group
    a.T = 256 / a.C1 < kProdGroups ? 256 / a.C1 : kProdGroups;
    if (a.T < 1) a.T = 1;
    const size_t stage = (size_t)a.T * 128 * KP * 2;
    a.stages = (int)((128 * 1024) / stage);
    if (a.stages > kMaxStages) a.stages = kMaxStages;
    if (a.stages < 2) return PPO_ERR_UNSUPPORTED;
    const size_t smem = (size_t)a.stages * stage + ((size_t)(a.C1 * KP * 2 + 1023) / 1024) * 1024 + sizeof(Pipe) + 1024;
    static bool attr_set[64] = {false};
    int dev = 0;
    PPO_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return PPO_ERR_CUDA;
    if (!attr_set[dev]) {
        PPO_CUDA_CHECK(cudaFuncSetAttribute(conv1_tc_kernel<KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        attr_set[dev] = true;
    }
    if (smem > 200 * 1024) return PPO_ERR_UNSUPPORTED;
    const int sms = ppo_num_sms();
    const int nstage = (a.tiles + a.T - 1) / a.T;
    conv1_tc_kernel<KS><<<nstage < sms ? nstage : sms, kThreads, smem, st>>>(a);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

}  // namespace

// out[m][co] = relu(bias[co] + sum_tap depth(m, tap) * W[co][tap]) as bf16; `bits` (optional, C1 % 32 == 0) gets the
// ReLU gates.  Returns PPO_ERR_UNSUPPORTED (nothing launched) for shapes it does not cover: C1 must be a multiple
// of 16 up to 256 (of 32 when bits are wanted), k in {3, 5, 7}.
int conv1_tc_fwd(const __half *depth, const bf16 *W, const float *bias, bf16 *out, uint32_t *bits, int rows, int Hi,
                 int Wi, int Ho, int Wo, int C1, int ks, int32_t *status, cudaStream_t st) {
    if (!status || C1 % 16 != 0 || C1 > 256 || C1 < 16 || (bits && C1 % 32 != 0)) return PPO_ERR_UNSUPPORTED;
    Args a;
    a.depth = depth; a.W = W; a.bias = bias; a.out = out; a.bits = bits;
    a.M = (long long)rows * Ho * Wo;
    a.Hi = Hi; a.Wi = Wi; a.Ho = Ho; a.Wo = Wo; a.C1 = C1;
    a.KP = (ks * ks + 15) / 16 * 16;
    const long long tiles = (a.M + 127) / 128;
    if (tiles <= 0) return PPO_OK;
    if (tiles > 0x7fffffffll) return PPO_ERR_UNSUPPORTED;
    a.tiles = (int)tiles;
    a.status = status;
    if (ks == 3) return launch<3>(a, st);
    if (ks == 5) return launch<5>(a, st);
    if (ks == 7) return launch<7>(a, st);
    return PPO_ERR_UNSUPPORTED;
}
