// Encoder forward/backward: the direct first convolution (C_in = 1), pooling, the small
// element-wise kernels, and the orchestration of the implicit GEMMs of the deeper layers.
#include "common.cuh"
#include "gemm.cuh"

// -------------------------------------------------------------------- conv1 ----

// First layer (C_in = 1): too shallow a reduction (k*k) for a tensor-core tile, and bound by
// HBM (reads one fp16 frame, writes C1 bf16 maps).  One thread per output pixel; the k*k
// patch sits in registers, the weights (as the bf16 shadow rounds them) in shared memory.
template <int KS>
__global__ void __launch_bounds__(128) conv1_fwd_kernel(const __half *__restrict__ depth,
                                                        const bf16 *__restrict__ W, const float *__restrict__ bias,
                                                        bf16 *__restrict__ out, int rows, int Hi, int Wi, int Ho,
                                                        int Wo, int C1) {
    extern __shared__ float sm[];  // w[tap][co], then bias[co]
    float *w = sm, *bs = sm + KS * KS * C1;
    for (int i = threadIdx.x; i < KS * KS * C1; i += blockDim.x) {
        const int co = i % C1, tap = i / C1;
        w[i] = bf2f(W[co * KS * KS + tap]);
    }
    for (int i = threadIdx.x; i < C1; i += blockDim.x) bs[i] = bias[i];
    __syncthreads();
    const long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long M = (long long)rows * Ho * Wo;
    if (m >= M) return;
    const int ow = (int)(m % Wo);
    const long long t = m / Wo;
    const int oh = (int)(t % Ho);
    const long long b = t / Ho;
    const __half *img = depth + b * Hi * Wi;
    constexpr int P = KS / 2;
    float x[KS * KS];
#pragma unroll
    for (int kh = 0; kh < KS; ++kh)
#pragma unroll
        for (int kw = 0; kw < KS; ++kw) {
            const int ih = 2 * oh + kh - P, iw = 2 * ow + kw - P;
            x[kh * KS + kw] = (ih >= 0 && ih < Hi && iw >= 0 && iw < Wi) ? __half2float(img[ih * Wi + iw]) : 0.f;
        }
    uint4 *o = reinterpret_cast<uint4 *>(out + m * C1);
    for (int c8 = 0; c8 < C1; c8 += 8) {
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = bs[c8 + j];
#pragma unroll
        for (int tap = 0; tap < KS * KS; ++tap)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = fmaf(w[tap * C1 + c8 + j], x[tap], acc[j]);
        __nv_bfloat162 p[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) p[j] = __floats2bfloat162_rn(fmaxf(acc[2 * j], 0.f), fmaxf(acc[2 * j + 1], 0.f));
        o[c8 / 8] = *reinterpret_cast<uint4 *>(p);
    }
}

// dW1[co][tap] += sum_m dZ1[m][co] * x(m, tap);  db1[co] += sum_m dZ1[m][co].
// A block stages TM output pixels (their gradients and input patches) in shared memory,
// then each thread owns a few (co, tap) pairs and reduces over the staged pixels.
template <int KS>
__global__ void __launch_bounds__(256) conv1_wgrad_kernel(const __half *__restrict__ depth,
                                                          const bf16 *__restrict__ dZ, float *__restrict__ dW,
                                                          float *__restrict__ db, int rows, int Hi, int Wi, int Ho,
                                                          int Wo, int C1) {
    constexpr int TM = 64, K2 = KS * KS, MAXP = 8;
    extern __shared__ float sm[];
    float *dz = sm;             // [TM][C1]
    float *px = sm + TM * C1;   // [TM][K2]
    const int npairs = C1 * K2 + C1;
    float acc[MAXP];
#pragma unroll
    for (int j = 0; j < MAXP; ++j) acc[j] = 0.f;
    const long long M = (long long)rows * Ho * Wo;
    constexpr int P = KS / 2;
    for (long long m0 = (long long)blockIdx.x * TM; m0 < M; m0 += (long long)gridDim.x * TM) {
        __syncthreads();
        for (int i = threadIdx.x; i < TM * C1; i += blockDim.x) {
            const long long m = m0 + i / C1;
            dz[i] = (m < M) ? bf2f(dZ[m * C1 + i % C1]) : 0.f;
        }
        for (int i = threadIdx.x; i < TM * K2; i += blockDim.x) {
            const int mm = i / K2, tap = i % K2;
            const long long m = m0 + mm;
            float v = 0.f;
            if (m < M) {
                const int ow = (int)(m % Wo);
                const long long t = m / Wo;
                const int oh = (int)(t % Ho);
                const long long b = t / Ho;
                const int ih = 2 * oh + tap / KS - P, iw = 2 * ow + tap % KS - P;
                if (ih >= 0 && ih < Hi && iw >= 0 && iw < Wi) v = __half2float(depth[(b * Hi + ih) * Wi + iw]);
            }
            px[i] = v;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < MAXP; ++j) {
            const int p = threadIdx.x + j * 256;
            if (p < npairs) {
                float s = 0.f;
                if (p < C1 * K2) {
                    const int co = p % C1, tap = p / C1;
#pragma unroll 8
                    for (int mm = 0; mm < TM; ++mm) s = fmaf(dz[mm * C1 + co], px[mm * K2 + tap], s);
                } else {
                    const int co = p - C1 * K2;
#pragma unroll 8
                    for (int mm = 0; mm < TM; ++mm) s += dz[mm * C1 + co];
                }
                acc[j] += s;
            }
        }
    }
#pragma unroll
    for (int j = 0; j < MAXP; ++j) {
        const int p = threadIdx.x + j * 256;
        if (p < C1 * K2) atomicAdd(dW + (p % C1) * K2 + p / C1, acc[j]);
        else if (p < npairs) atomicAdd(db + (p - C1 * K2), acc[j]);
    }
}

// ------------------------------------------------------------- small kernels ----

// h0[b] = [mean over pixels of act[b][px][c], proprio[b]] as bf16.  One block per row b.
__global__ void __launch_bounds__(256) pool_concat_kernel(const bf16 *__restrict__ act,
                                                          const float *__restrict__ proprio, bf16 *__restrict__ h0,
                                                          int npx, int C, int P) {
    const int b = blockIdx.x;
    const float inv = 1.f / (float)npx;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const bf16 *p = act + (size_t)b * npx * C + c;
        float s = 0.f;
        for (int px = 0; px < npx; ++px) s += bf2f(p[(size_t)px * C]);
        h0[(size_t)b * (C + P) + c] = __float2bfloat16_rn(s * inv);
    }
    for (int j = threadIdx.x; j < P; j += blockDim.x)
        h0[(size_t)b * (C + P) + C + j] = __float2bfloat16_rn(proprio[(size_t)b * P + j]);
}

// dact[b][px][c] = dh0[b][c] / npx where act > 0, else 0.
__global__ void __launch_bounds__(256) unpool_kernel(const float *__restrict__ dh0, const bf16 *__restrict__ act,
                                                     bf16 *__restrict__ dact, long long total, int npx, int C,
                                                     int ld_h0) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int c = (int)(i % C);
    const long long b = i / ((long long)npx * C);
    const float g = dh0[b * ld_h0 + c] / (float)npx;
    dact[i] = __float2bfloat16_rn(bf2f(act[i]) > 0.f ? g : 0.f);
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

// db[n] += sum_m dZ[m][n]  (bias gradients).  32 columns x 8 row groups per block.
__global__ void __launch_bounds__(256) colsum_kernel(const bf16 *__restrict__ dZ, int ld, long long M, int N,
                                                     float *__restrict__ db, int rows_per_block) {
    __shared__ float sh[8][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const long long m_lo = (long long)blockIdx.x * rows_per_block;
    const long long m_hi = min(M, m_lo + rows_per_block);
    for (int n0 = 0; n0 < N; n0 += 32) {
        const int n = n0 + tx;
        float s = 0.f;
        if (n < N)
            for (long long m = m_lo + ty; m < m_hi; m += 8) s += bf2f(dZ[m * ld + n]);
        sh[ty][tx] = s;
        __syncthreads();
        if (ty == 0 && n < N) {
            float t = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) t += sh[j][tx];
            atomicAdd(db + n, t);
        }
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
    if (m->impl == 1) return simt_gemm_fwd(g, X, W, e, st);
    return tc_gemm_fwd(g, X, W, e, ppo_device_status_ptr(), st);
}

static int run_dgrad(const ppo_model *m, const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *W, const bf16 *Wt,
                     int wt_ld, const DgradEpilogue &e, cudaStream_t st) {
    if (m->impl == 1) return simt_gemm_dgrad(g, dY, ldy, W, e, st);
    return tc_gemm_dgrad(g, dY, ldy, Wt, wt_ld, e, ppo_device_status_ptr(), st);
}

static int run_wgrad(const ppo_model *m, const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW,
                     cudaStream_t st) {
    if (m->impl == 1) return simt_gemm_wgrad(g, dY, ldy, X, dW, st);
    return tc_gemm_wgrad(g, dY, ldy, X, dW, ppo_device_status_ptr(), st);
}

static int run_colsum(const bf16 *dZ, int ld, long long M, int N, float *db, cudaStream_t st) {
    const int rpb = 512;
    colsum_kernel<<<ppo_cdiv(M, rpb), 256, 0, st>>>(dZ, ld, M, N, db, rpb);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

#define PPO_TRY(expr)                 \
    do {                              \
        int _s = (expr);              \
        if (_s != PPO_OK) return _s;  \
    } while (0)

static int check_rows(const ppo_model *m, const ppo_minibatch *mb, int row0, int rows) {
    if (!m || !mb) return PPO_ERR_INVALID_ARG;
    if (!m->master) return PPO_ERR_STATE;
    if (row0 < 0 || rows <= 0 || row0 + rows > mb->B || rows > m->mbmax) return PPO_ERR_SHAPE;
    if (!mb->depth_f16 || !mb->proprio) return PPO_ERR_INVALID_ARG;
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
        const size_t smem = (size_t)(KS * KS * C1 + C1) * sizeof(float);
        const bf16 *W = m->shadow + m->tensors[0].off;
        const float *bias = m->master + m->tensors[1].off;
        const int blocks = ppo_cdiv(M, 128);
#define PPO_CONV1(KS_)                                                                                            \
    conv1_fwd_kernel<KS_><<<blocks, 128, smem, st>>>(depth, W, bias, m->act[1], rows, d.H, d.W, m->Hs[1], m->Ws[1], C1)
        if (KS == 1) PPO_CONV1(1);
        else if (KS == 3) PPO_CONV1(3);
        else if (KS == 5) PPO_CONV1(5);
        else PPO_CONV1(7);
#undef PPO_CONV1
        PPO_LAUNCH_CHECK();
    }
    for (int l = 2; l <= m->L; ++l) {
        ConvGeom g = conv_geom(m, l, rows);
        FwdEpilogue e = {m->master + m->tensors[2 * (l - 1) + 1].off, 1, m->act[l], nullptr, nullptr, 0};
        PPO_TRY(run_fwd(m, g, m->act[l - 1], m->shadow + m->tensors[2 * (l - 1)].off, e, st));
    }
    pool_concat_kernel<<<rows, 256, 0, st>>>(m->act[m->L], mb->proprio + (size_t)row0 * d.P, m->h[0],
                                             m->Hs[m->L] * m->Ws[m->L], m->Cs[m->L], d.P);
    PPO_LAUNCH_CHECK();
    int ti = 2 * m->L;
    for (int l = 1; l <= m->F; ++l, ti += 2) {
        ConvGeom g = fc_geom(rows, m->hw[l - 1], m->hw[l]);
        FwdEpilogue e = {m->master + m->tensors[ti + 1].off, 1, m->h[l], nullptr, nullptr, 0};
        PPO_TRY(run_fwd(m, g, m->h[l - 1], m->shadow + m->tensors[ti].off, e, st));
    }
    {
        ConvGeom g = fc_geom(rows, m->hw[m->F], d.A + 1);
        FwdEpilogue e = {m->master + m->tensors[ti + 1].off, 0, nullptr, mean, value, d.A};
        PPO_TRY(run_fwd(m, g, m->h[m->F], m->shadow + m->tensors[ti].off, e, st));
    }
    m->fwd_valid = true;
    m->last_row0 = row0;
    m->last_rows = rows;
    return PPO_OK;
}

static int wt_ld_of(int Co) { return (Co + 7) / 8 * 8; }

static int refresh_transposed(ppo_model *m, cudaStream_t st) {
    if (m->wT_valid) return PPO_OK;
    for (int l = 2; l <= m->L; ++l) {
        const int Co = m->Cs[l], Ci = m->Cs[l - 1], taps = m->d.conv_k[l - 1] * m->d.conv_k[l - 1];
        const long long total = (long long)Ci * taps * wt_ld_of(Co);
        transpose_weights_kernel<<<ppo_cdiv(total, 256), 256, 0, st>>>(m->shadow + m->tensors[2 * (l - 1)].off,
                                                                     m->wT + m->wT_off[2 * (l - 1)], Co, taps, Ci,
                                                                     wt_ld_of(Co));
        PPO_LAUNCH_CHECK();
    }
    int ti = 2 * m->L;
    for (int l = 1; l <= m->F + 1; ++l, ti += 2) {
        const int Ci = m->hw[l - 1], Co = (l <= m->F) ? m->hw[l] : m->d.A + 1;
        const long long total = (long long)Ci * wt_ld_of(Co);
        transpose_weights_kernel<<<ppo_cdiv(total, 256), 256, 0, st>>>(m->shadow + m->tensors[ti].off,
                                                                     m->wT + m->wT_off[ti], Co, 1, Ci, wt_ld_of(Co));
        PPO_LAUNCH_CHECK();
    }
    m->wT_valid = true;
    return PPO_OK;
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
        PPO_CUDA_CHECK(cudaMemsetAsync(m->grad, 0, (size_t)m->tensors.back().off * sizeof(float), st));
    if (m->impl == 0) PPO_TRY(refresh_transposed(m, st));

    pack_dout_kernel<<<ppo_cdiv((long long)rows * 16, 256), 256, 0, st>>>(dmean, dvalue, m->dh[F + 1], rows, d.A);
    PPO_LAUNCH_CHECK();
    // head and hidden FC layers, last to first; layer index F+1 is the head
    for (int l = F + 1; l >= 1; --l) {
        const int ti = 2 * L + 2 * (l - 1);
        const int Co = (l <= F) ? m->hw[l] : d.A + 1;
        const int ldy = (l <= F) ? Co : 16;
        ConvGeom g = fc_geom(rows, m->hw[l - 1], Co);
        const bf16 *dY = m->dh[l];
        PPO_TRY(run_wgrad(m, g, dY, ldy, m->h[l - 1], m->grad + m->tensors[ti].off, st));
        PPO_TRY(run_colsum(dY, ldy, rows, Co, m->grad + m->tensors[ti + 1].off, st));
        DgradEpilogue e;
        if (l > 1) e = {m->h[l - 1], m->dh[l - 1], nullptr};
        else e = {nullptr, nullptr, m->dh0_f32};
        PPO_TRY(run_dgrad(m, g, dY, ldy, m->shadow + m->tensors[ti].off, m->wT + m->wT_off[ti], wt_ld_of(Co), e, st));
    }
    {
        const int npx = m->Hs[L] * m->Ws[L], C = m->Cs[L];
        const long long total = (long long)rows * npx * C;
        unpool_kernel<<<ppo_cdiv(total, 256), 256, 0, st>>>(m->dh0_f32, m->act[L], m->dact[L], total, npx, C,
                                                          m->hw[0]);
        PPO_LAUNCH_CHECK();
    }
    for (int l = L; l >= 2; --l) {
        const int ti = 2 * (l - 1);
        ConvGeom g = conv_geom(m, l, rows);
        PPO_TRY(run_wgrad(m, g, m->dact[l], g.Co, m->act[l - 1], m->grad + m->tensors[ti].off, st));
        PPO_TRY(run_colsum(m->dact[l], g.Co, g.M(), g.Co, m->grad + m->tensors[ti + 1].off, st));
        DgradEpilogue e = {m->act[l - 1], m->dact[l - 1], nullptr};
        PPO_TRY(run_dgrad(m, g, m->dact[l], g.Co, m->shadow + m->tensors[ti].off, m->wT + m->wT_off[ti],
                          wt_ld_of(g.Co), e, st));
    }
    {   // conv1: weight and bias gradients only
        const __half *depth = static_cast<const __half *>(mb->depth_f16) + (size_t)row0 * d.H * d.W;
        const int C1 = m->Cs[1], KS = d.conv_k[0];
        const long long M = (long long)rows * m->Hs[1] * m->Ws[1];
        const size_t smem = (size_t)64 * (C1 + KS * KS) * sizeof(float);
        int blocks = ppo_cdiv(M, 64);
        const int cap = ppo_num_sms() * 4;
        if (blocks > cap) blocks = cap;
        float *dW = m->grad + m->tensors[0].off, *db = m->grad + m->tensors[1].off;
#define PPO_CONV1W(KS_)                                                                                       \
    conv1_wgrad_kernel<KS_><<<blocks, 256, smem, st>>>(depth, m->dact[1], dW, db, rows, d.H, d.W, m->Hs[1], \
                                                       m->Ws[1], C1)
        if (KS == 1) PPO_CONV1W(1);
        else if (KS == 3) PPO_CONV1W(3);
        else if (KS == 5) PPO_CONV1W(5);
        else PPO_CONV1W(7);
#undef PPO_CONV1W
        PPO_LAUNCH_CHECK();
    }
    return PPO_OK;
}
