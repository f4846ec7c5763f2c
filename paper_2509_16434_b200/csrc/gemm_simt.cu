// CUDA-core reference versions of the encoder's implicit GEMMs: a plain 64x64x16 shared
// memory tiling with functors for the operand gathers.  Same operand precision as the
// tensor-core kernels (bf16 operands, fp32 accumulation); selected with
// PPO_B200_ENCODER=simt as a debugging aid.
#include "gemm.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

// C[m][n] = sum_k a(m, k) * b(k, n) over k in [k0, k1); epi(m, n, acc) for m < M, n < N.
template <class AF, class BF, class Epi>
__global__ void __launch_bounds__(256) simt_gemm_kernel(long long M, int N, long long K, long long k_per_split,
                                                        AF a, BF b, Epi epi) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const long long m0 = (long long)blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;
    const long long k0 = (long long)blockIdx.z * k_per_split;
    const long long k1 = min(K, k0 + k_per_split);
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (long long kb = k0; kb < k1; kb += BK) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = threadIdx.x + e * 256;
            {   // A tile: k fastest so that consecutive threads read consecutive k of one row
                const int kk = idx % BK, mm = idx / BK;
                const long long m = m0 + mm, k = kb + kk;
                As[kk][mm] = (m < M && k < k1) ? a(m, k) : 0.f;
            }
            {   // B tile: n fastest
                const int nn = idx % BN, kk = idx / BN;
                const int n = n0 + nn;
                const long long k = kb + kk;
                Bs[kk][nn] = (n < N && k < k1) ? b(k, n) : 0.f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long long m = m0 + ty * 4 + i;
            const int n = n0 + tx * 4 + j;
            if (m < M && n < N) epi(m, n, acc[i][j]);
        }
}

struct Im2col {  // (m, k=(tap,ci)) -> X[b, 2oh+kh-p, 2ow+kw-p, ci]
    const bf16 *X;
    ConvGeom g;
    __device__ float operator()(long long m, long long k) const {
        const int ci = (int)(k % g.Ci), tap = (int)(k / g.Ci);
        const int kw = tap % g.k, kh = tap / g.k;
        const int ow = (int)(m % g.Wo);
        const long long t = m / g.Wo;
        const int oh = (int)(t % g.Ho);
        const long long b = t / g.Ho;
        const int ih = 2 * oh + kh - g.pad, iw = 2 * ow + kw - g.pad;
        if (ih < 0 || ih >= g.Hi || iw < 0 || iw >= g.Wi) return 0.f;
        return bf2f(X[((b * g.Hi + ih) * g.Wi + iw) * g.Ci + ci]);
    }
};

struct WeightKN {  // (k, n=co) -> W[co][k]
    const bf16 *W;
    int K;
    __device__ float operator()(long long k, int n) const { return bf2f(W[(size_t)n * K + k]); }
};

struct FwdEpi {
    FwdEpilogue e;
    int Co;
    __device__ void operator()(long long m, int n, float acc) const {
        float v = acc + e.bias[n];
        if (e.relu) v = fmaxf(v, 0.f);
        if (e.out) e.out[m * Co + n] = __float2bfloat16_rn(v);
        else if (n < e.A) e.out_mean[m * e.A + n] = v;
        else e.out_value[m] = v;
    }
};

struct DyGather {  // (m'=(b,ih,iw), k=(tap,co)) -> dY[b, (ih+p-kh)/2, (iw+p-kw)/2, co]
    const bf16 *dY;
    int ldy;
    ConvGeom g;
    __device__ float operator()(long long m, long long k) const {
        const int co = (int)(k % g.Co), tap = (int)(k / g.Co);
        const int kw = tap % g.k, kh = tap / g.k;
        const int iw = (int)(m % g.Wi);
        const long long t = m / g.Wi;
        const int ih = (int)(t % g.Hi);
        const long long b = t / g.Hi;
        const int th = ih + g.pad - kh, tw = iw + g.pad - kw;
        if (th < 0 || tw < 0 || (th & 1) || (tw & 1)) return 0.f;
        const int oh = th >> 1, ow = tw >> 1;
        if (oh >= g.Ho || ow >= g.Wo) return 0.f;
        return bf2f(dY[((b * g.Ho + oh) * g.Wo + ow) * ldy + co]);
    }
};

struct WeightDgrad {  // (k=(tap,co), n=ci) -> W[co][tap][ci]
    const bf16 *W;
    ConvGeom g;
    __device__ float operator()(long long k, int n) const {
        const int co = (int)(k % g.Co), tap = (int)(k / g.Co);
        return bf2f(W[((size_t)co * g.taps() + tap) * g.Ci + n]);
    }
};

struct DgradEpi {
    DgradEpilogue e;
    int Ci;
    __device__ void operator()(long long m, int n, float acc) const {
        float v = acc;
        if (e.mask_act && !(bf2f(e.mask_act[m * Ci + n]) > 0.f)) v = 0.f;
        if (e.out) e.out[m * Ci + n] = __float2bfloat16_rn(v);
        if (e.out_f32) e.out_f32[m * Ci + n] = v;
    }
};

struct DyT {  // (m''=co, k=m) -> dY[m][co]
    const bf16 *dY;
    int ldy;
    __device__ float operator()(long long co, long long m) const { return bf2f(dY[m * ldy + co]); }
};

struct Im2colKN {  // (k=m, n=(tap,ci))
    Im2col f;
    __device__ float operator()(long long m, int n) const { return f(m, n); }
};

struct WgradEpi {
    float *dW;
    int K;
    __device__ void operator()(long long co, int n, float acc) const { atomicAdd(dW + co * K + n, acc); }
};

}  // namespace

int simt_gemm_fwd(const ConvGeom &g, const bf16 *X, const bf16 *W, const FwdEpilogue &e, cudaStream_t st) {
    const long long M = g.M();
    dim3 grid(ppo_cdiv(M, BM), ppo_cdiv(g.Co, BN), 1);
    simt_gemm_kernel<<<grid, 256, 0, st>>>(M, g.Co, (long long)g.K(), (long long)g.K(), Im2col{X, g},
                                           WeightKN{W, g.K()}, FwdEpi{e, g.Co});
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

int simt_gemm_dgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *W, const DgradEpilogue &e,
                    cudaStream_t st) {
    const long long M = (long long)g.B * g.Hi * g.Wi;
    const long long K = (long long)g.taps() * g.Co;
    dim3 grid(ppo_cdiv(M, BM), ppo_cdiv(g.Ci, BN), 1);
    simt_gemm_kernel<<<grid, 256, 0, st>>>(M, g.Ci, K, K, DyGather{dY, ldy, g}, WeightDgrad{W, g}, DgradEpi{e, g.Ci});
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

int simt_gemm_wgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW, cudaStream_t st) {
    const long long K = g.M();
    const int N = g.K();
    const int tiles = ppo_cdiv(g.Co, BM) * ppo_cdiv(N, BN);
    // split the long reduction so that a few waves of CTAs are in flight
    long long splits = (long long)ppo_num_sms() * 4 / tiles;
    if (splits < 1) splits = 1;
    long long per = (K + splits - 1) / splits;
    per = (per + BK - 1) / BK * BK;
    if (per < 4 * BK) per = 4 * BK;
    splits = (K + per - 1) / per;
    dim3 grid(ppo_cdiv(g.Co, BM), ppo_cdiv(N, BN), (unsigned)splits);
    simt_gemm_kernel<<<grid, 256, 0, st>>>((long long)g.Co, N, K, per, DyT{dY, ldy}, Im2colKN{Im2col{X, g}},
                                           WgradEpi{dW, N});
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}
