// First convolution (one input channel) on the tensor cores.
//
// Per output pixel the layer is a dot product of k*k depth values with each of C1 filters: far too short a
// reduction for the CUDA cores to do cheaply (C1 * k*k multiply-adds per pixel, one instruction each), but
// one tcgen05.mma of K = 16 covers a 3x3 window for 128 pixels and all filters at once.  Producer threads
// build the im2col tile themselves, one pixel per thread, directly in the unswizzled K-major core-matrix
// layout (8 rows x 16 bytes per core matrix).  A window row starts at an even or odd column of the frame, so
// the thread fetches it as aligned pairs of fp16 pixels (32-bit loads) and stores the pairs as they are: the
// K axis is laid out as (window row, pair, element of the pair), with one element per row that lies outside
// the window and meets a zero filter entry.  Nothing is unpacked or repacked, so the producer is a stream of
// loads and stores.  The filters are converted from the bf16 shadow to fp16 once per CTA, so that both
// operands are fp16 and the depth values enter exactly; the bias rides in two spare K slots as a pair of fp16
// values (high part, remainder) against a constant 1.  fp32 accumulation in tensor memory; the epilogue is
// ReLU + bf16 conversion in one instruction per pair, the one-bit ReLU gates the backward pass reads, and a
// pass through shared memory so that every store instruction of a warp writes contiguous bytes.
// Frames must hold finite values (an Inf or NaN beside a window would meet a zero weight) and have an even
// width.
#include "gemm.cuh"
#include "tcgen05.cuh"

namespace {

using namespace tc;

constexpr int kMaxStages = 8;
constexpr int kProdWarps = 4;    // 128 producer threads; thread r fills row r of every tile of a stage with asynchronous copies
constexpr int kMaxT = 5;         // tiles per stage at most
constexpr int kEpiWarps = 20;    // five per TMEM lane quarter, which take the column groups in turn
constexpr int kThreads = (kProdWarps + 1 + kEpiWarps) * 32;

struct Args {
    const __half *depth;
    const bf16 *W;      // [C1][k*k] bf16
    const float *bias;  // [C1]
    bf16 *out;          // [M][C1]
    uint32_t *bits;     // [M][C1 / 32] or null
    const float *ln_gamma, *ln_beta;  // layer normalisation over the C1 channels of a pixel (null: none; C1 = 16 or 32)
    bf16 *ln_xhat;      // [M][C1]
    float *ln_rstd;     // [M]
    long long M;        // output pixels
    int Hi, Wi, Ho, Wo, C1;
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
    alignas(16) float gamma[32], beta[32];
};

// Unswizzled K-major operand image: element (row r, column k) of a tile with KP columns lives at
// (r / 8) * (KP / 8) * 128 + (k / 8) * 128 + (r % 8) * 16 + (k % 8) * 2 bytes.
__device__ __forceinline__ uint32_t core_offset(int r, int kchunk, int KP) {
    return (uint32_t)(r >> 3) * (uint32_t)(KP >> 3) * 128u + (uint32_t)kchunk * 128u + (uint32_t)(r & 7) * 16u;
}

// Four bytes global -> shared without passing through registers; !valid writes zeros (no source byte is read).
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src, bool valid) {
    const uint32_t n = valid ? 4u : 0u;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}

__device__ __forceinline__ uint64_t desc_nosw(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

// kind::f16 with fp16 A and B (format 0), fp32 D, both K-major.
__host__ __device__ constexpr uint32_t idesc_f16(int M, int N) {
    return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// K layout of a window of size KS: window row kh holds NP pairs; pair q covers frame columns
// 2 ow - P - ODD + 2 q (+1), element e of it is kernel column 2 q + e - ODD (outside 0 .. KS-1: zero filter entry).
// Halves 2 KS NP and 2 KS NP + 1 carry the constant 1 for the two bias parts; the rest up to KP are zero.
template <int KS>
struct Win {
    static constexpr int P = KS / 2, ODD = P & 1, NP = (KS + ODD + 1) / 2;
    static constexpr int KW = KS * NP;                     // 32-bit words of window data
    static constexpr int KP = (2 * KW + 2 + 15) / 16 * 16; // halves per im2col row
};

template <int KS>
__global__ void __launch_bounds__(kThreads, 1) conv1_tc_kernel(const __grid_constant__ Args a) {
    using WN = Win<KS>;
    constexpr int K2 = KS * KS, KP = WN::KP, P = WN::P, ODD = WN::ODD, NP = WN::NP, KW = WN::KW;
    constexpr uint32_t kTileBytes = 128u * KP * 2u;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int N = a.C1, T = a.T, S = a.stages;
    const uint32_t stage_bytes = (uint32_t)T * kTileBytes;
    uint8_t *bsm = smem + (size_t)S * stage_bytes;                 // filters [N][KP] fp16
    Pipe *pipe = reinterpret_cast<Pipe *>(bsm + ((N * KP * 2 + 1023) / 1024) * 1024);
    uint4 *staging = reinterpret_cast<uint4 *>(pipe + 1);          // per epilogue warp 32 pixels x 64 bytes
    volatile int *abort_flag = &pipe->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t acc_cols = tmem_cols_for(T * N);                // T accumulators side by side
    const int nacc_log = acc_cols * 4 <= 512 ? 2 : 1, nacc = 1 << nacc_log;
    const uint32_t ncols = acc_cols * nacc;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe->full[s], kProdWarps * 32);
            mbar_init(&pipe->empty[s], 1);
        }
        for (int i = 0; i < nacc; ++i) {
            mbar_init(&pipe->tfull[i], 1);
            mbar_init(&pipe->tempty[i], kEpiWarps * 32);
        }
        pipe->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // filters in the K layout of the window, bias parts in the two slots behind it, zeros elsewhere
    for (int i = threadIdx.x; i < N * KP; i += kThreads) {
        const int n = i / KP, k = i - n * KP;
        float f = 0.f;
        if (k < 2 * KW) {
            const int w = k >> 1, kh = w / NP, kw = 2 * (w - kh * NP) + (k & 1) - ODD;
            if (kw >= 0 && kw < KS) f = bf2f(a.W[n * K2 + kh * KS + kw]);
        } else if (k == 2 * KW) {
            f = __half2float(__float2half_rn(a.bias[n]));
        } else if (k == 2 * KW + 1) {
            f = a.bias[n] - __half2float(__float2half_rn(a.bias[n]));
        }
        *reinterpret_cast<__half *>(bsm + core_offset(n, k >> 3, KP) + (k & 7) * 2) = __float2half_rn(f);
    }
    // The constant part of every im2col row of every stage: the two bias slots hold 1.0 (as fp16), the padding behind
    // them zero.  The producers' copies only ever write the window words in front of it.
    for (int i = threadIdx.x; i < S * T * 128; i += kThreads) {
        uint8_t *row = smem + (size_t)(i >> 7) * kTileBytes;
#pragma unroll
        for (int k = KW; k < KP / 2; ++k)
            *reinterpret_cast<uint32_t *>(row + core_offset(i & 127, k >> 2, KP) + (k & 3) * 4) = k == KW ? 0x3C003C00u : 0u;
    }
    if (a.ln_gamma && threadIdx.x < 32) {
        pipe->gamma[threadIdx.x] = (int)threadIdx.x < N ? a.ln_gamma[threadIdx.x] : 0.f;
        pipe->beta[threadIdx.x] = (int)threadIdx.x < N ? a.ln_beta[threadIdx.x] : 0.f;
    }
    fence_async_smem();
    if (warp == kProdWarps) tmem_alloc(&pipe->tmem_slot, ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = pipe->tmem_slot;
    const uint32_t smem_base = smem_u32(smem);

    // contiguous run of stages (T tiles each) for this CTA
    const int nstage_all = (a.tiles + T - 1) / T;
    const int q = nstage_all / (int)gridDim.x, rem = nstage_all - q * (int)gridDim.x, b = (int)blockIdx.x;
    const int s0 = b * q + (b < rem ? b : rem), ns = q + (b < rem ? 1 : 0);

    if (warp < kProdWarps) {
        // ---------------- producers: thread r owns row r of each of the stage's T tiles.  A window goes from the frame
        // straight into its im2col row as aligned pairs of fp16 pixels, one 4-byte asynchronous copy per pair (zeros
        // where the pair lies outside the frame or the pixel past the end); the copies of up to S stages are in flight
        // while the thread moves on, and the stage's barrier counts them in as they land.
        const int r = threadIdx.x;
        bool ok = true;
        const int hw = a.Ho * a.Wo;
        const int d_b = 128 / hw, d_oh = (128 % hw) / a.Wo, d_ow = 128 % a.Wo;  // 128 pixels further, without divisions
        const int Wh = a.Wi >> 1;  // 32-bit words per frame row
        const uint32_t *frames = reinterpret_cast<const uint32_t *>(a.depth);
        long long m = (long long)s0 * T * 128 + r;
        int ow = (int)(m % a.Wo);
        int oh, ib;
        {
            const long long t = m / a.Wo;
            oh = (int)(t % a.Ho);
            ib = (int)(t / a.Ho);
        }
        const uint32_t row_off = core_offset(r, 0, KP);
        int s = 0;
        uint32_t ph = 0;
        for (int li = 0; li < ns && ok; ++li) {
            ok = mbar_wait(&pipe->empty[s], ph ^ 1u, abort_flag, a.status);
            if (!ok) break;
            uint32_t dst = smem_base + (uint32_t)s * stage_bytes + row_off;
            for (int g = 0; g < T; ++g, dst += kTileBytes) {
                const bool live = m < a.M;
                const uint32_t *img = frames + (long long)(live ? ib : 0) * a.Hi * Wh;
                const int pw0 = ow - (P + ODD) / 2;  // first pair of the window row, in words
#pragma unroll
                for (int kh = 0; kh < KS; ++kh) {
                    const int ih = 2 * oh + kh - P;
                    const bool rok = live && (unsigned)ih < (unsigned)a.Hi;
                    const uint32_t *row = img + (rok ? ih : 0) * Wh;
#pragma unroll
                    for (int qq = 0; qq < NP; ++qq) {
                        const int pw = pw0 + qq, k = kh * NP + qq;
                        const bool pok = rok && (unsigned)pw < (unsigned)Wh;
                        cp_async4(dst + (uint32_t)(k >> 2) * 128u + (uint32_t)(k & 3) * 4u, row + (pok ? pw : 0), pok);
                    }
                }
                m += 128;
                ow += d_ow;
                if (ow >= a.Wo) { ow -= a.Wo; ++oh; }
                oh += d_oh;
                if (oh >= a.Ho) { oh -= a.Ho; ++ib; }
                ib += d_b;
            }
            cp_async_arrive(&pipe->full[s]);
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        cp_async_wait<0>();
    } else if (warp == kProdWarps) {
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
            fence_async_smem();  // the producers' copies were ordinary shared-memory writes; the tensor core reads through the async proxy
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
        // ---------------- epilogue: TMEM lane = pixel of a tile; warp w reads lanes 32 (w % 4) .. +31; the
        // warps of a lane quarter take the groups of 32 accumulator columns in turn (16 when C1 is not a multiple
        // of 32)
        const int ew = warp - (kProdWarps + 1), lg = warp & 3, half = ew >> 2;
        const int p = lg * 32 + lane;
        const int CW = (N & 31) == 0 ? 32 : 16;
        uint4 *stg = staging + (size_t)ew * 128;
        const int sw = (lane >> 1) & 3, rr0 = lane >> 2, piece = lane & 3;
        bool ok = true;
        for (int li = 0; li < ns && ok; ++li) {
            const int acc = li & (nacc - 1);
            ok = mbar_wait(&pipe->tfull[acc], (li >> nacc_log) & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t lane_base = tmem_base + acc * acc_cols + ((uint32_t)(lg * 32) << 16);
            for (int cc = half * CW; cc < T * N; cc += (kEpiWarps / 4) * CW) {   // column of the accumulator: tile g, channel c0
                const int g = cc / N, c0 = cc - g * N;
                const long long m0 = ((long long)(s0 + li) * T + g) * 128 + lg * 32;  // first pixel of this warp
                float v[32];
                tmem_ld16(lane_base + (uint32_t)cc, v);
                if (CW == 32) tmem_ld16(lane_base + (uint32_t)cc + 16u, v + 16);
                uint32_t pk[16];
                uint32_t gate = 0;
                if (a.ln_gamma) {
                    // layer normalisation over the CW = C1 channels this thread holds: two passes in registers; the
                    // normalised values are stored pixel by pixel (a thread's CW values are contiguous)
                    float sum = 0.f, sq = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < CW) sum += v[i];
                    const float mean = sum / (float)CW;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < CW) sq += (v[i] - mean) * (v[i] - mean);
                    const float rs = rsqrtf(sq / (float)CW + kLnEps);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < CW) v[i] = (v[i] - mean) * rs;
                    if (m0 + lane < a.M) {
                        uint4 *xp = reinterpret_cast<uint4 *>(a.ln_xhat + (m0 + lane) * N + c0);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (j < CW / 8)
                                xp[j] = make_uint4(pack_bf16x2(v[8 * j], v[8 * j + 1]), pack_bf16x2(v[8 * j + 2], v[8 * j + 3]),
                                                   pack_bf16x2(v[8 * j + 4], v[8 * j + 5]), pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
                        a.ln_rstd[m0 + lane] = rs;
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < CW) v[i] = fmaf(pipe->gamma[c0 + i], v[i], pipe->beta[c0 + i]);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (j < CW / 2) {
                        pk[j] = relu_pack_bf16x2(v[2 * j], v[2 * j + 1]);
                        gate = gate_bits_add(gate, pk[j], j);
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < CW / 8) stg[lane * 4 + (j ^ sw)] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                if (a.bits && m0 + lane < a.M) a.bits[(m0 + lane) * (N >> 5) + (c0 >> 5)] = gate;
                __syncwarp();
#pragma unroll
                for (int ps = 0; ps < 4; ++ps) {
                    const int rr = ps * 8 + rr0;
                    if (m0 + rr < a.M && piece < CW / 8)
                        *reinterpret_cast<uint4 *>(a.out + (m0 + rr) * N + c0 + piece * 8) = stg[rr * 4 + (piece ^ ((rr >> 1) & 3))];
                }
                __syncwarp();
            }
            tc_fence_before();
            mbar_arrive(&pipe->tempty[acc]);
        }
        (void)p;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProdWarps) {
        tc_fence_after();
        tmem_dealloc(tmem_base, ncols);
    }
}

template <int KS>
int launch(Args &a, cudaStream_t st) {
    constexpr int KP = Win<KS>::KP;
    // tiles per stage: as many accumulators as fit twice into the 512 columns of tensor memory, at most kMaxT
    a.T = 256 / a.C1 < kMaxT ? 256 / a.C1 : kMaxT;
    if (a.T < 1) a.T = 1;
    const size_t stage = (size_t)a.T * 128 * KP * 2;
    a.stages = (int)((128 * 1024) / stage);
    if (a.stages > kMaxStages) a.stages = kMaxStages;
    if (a.stages < 2) return PPO_ERR_UNSUPPORTED;
    const size_t smem = (size_t)a.stages * stage + ((size_t)(a.C1 * KP * 2 + 1023) / 1024) * 1024 + sizeof(Pipe) +
                        (size_t)kEpiWarps * 2048 + 1024;
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
// of 16 up to 256 (of 32 when bits are wanted), k in {3, 5, 7}, the frame width even and the frames 4-byte aligned.
int conv1_tc_fwd(const __half *depth, const bf16 *W, const float *bias, bf16 *out, uint32_t *bits, int rows, int Hi,
                 int Wi, int Ho, int Wo, int C1, int ks, const float *ln_gamma, const float *ln_beta, bf16 *ln_xhat,
                 float *ln_rstd, int32_t *status, cudaStream_t st) {
    if (!status || C1 % 16 != 0 || C1 > 256 || C1 < 16 || (bits && C1 % 32 != 0)) return PPO_ERR_UNSUPPORTED;
    if (ln_gamma && ((C1 != 16 && C1 != 32) || !ln_beta || !ln_xhat || !ln_rstd)) return PPO_ERR_UNSUPPORTED;
    if (Wi % 2 != 0 || !ppo_aligned(depth, 4)) return PPO_ERR_UNSUPPORTED;
    Args a;
    a.depth = depth; a.W = W; a.bias = bias; a.out = out; a.bits = bits;
    a.ln_gamma = ln_gamma; a.ln_beta = ln_beta; a.ln_xhat = ln_xhat; a.ln_rstd = ln_rstd;
    a.M = (long long)rows * Ho * Wo;
    a.Hi = Hi; a.Wi = Wi; a.Ho = Ho; a.Wo = Wo; a.C1 = C1;
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
