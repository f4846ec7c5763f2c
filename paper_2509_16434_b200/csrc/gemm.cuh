// The three GEMM-shaped operations of the encoder, as implicit GEMMs over NHWC bf16
// activations.  A fully connected layer is the case Hi = Wi = Ho = Wo = 1, k = 1, pad = 0.
//   fwd   : Y[m][co]  = act( bias[co] + sum_{tap,ci} X[b, 2oh+kh-p, 2ow+kw-p, ci] * W[co][tap][ci] )
//   dgrad : dX[m'][ci] = mask( sum_{tap,co} dY[b, (ih+p-kh)/2, (iw+p-kw)/2, co] * W[co][tap][ci] )
//   wgrad : dW[co][tap][ci] += sum_m dY[m][co] * X[b, 2oh+kh-p, 2ow+kw-p, ci]
// m = (b, oh, ow) over output pixels, m' = (b, ih, iw) over input pixels; fp32 accumulation.
#pragma once
#include "common.cuh"

struct FwdEpilogue {
    const float *bias;  // [Co] fp32
    int relu;
    bf16 *out;          // [M][Co] bf16, or nullptr when the head outputs below are used
    float *out_mean;    // head: columns 0..A-1 -> [M][A]
    float *out_value;   // head: column A -> [M]
    int A;
    uint32_t *out_bits = nullptr;  // optional: gate bits (out > 0) of a ReLU output, [M][Co / 32]; needs Co % 32 == 0
    int ldo = 0;                   // row stride of `out` in elements (0: Co)
    // Layer normalisation over the Co channels of every output row, between the bias and the ReLU (all null: none):
    // xhat = (z - mean) / sqrt(var + 1e-5), out = act(gamma * xhat + beta); xhat [M][Co] bf16 and rstd [M] fp32 are
    // kept for the backward pass.  Needs Co <= 256 (one column tile) and ldo == Co.
    const float *ln_gamma = nullptr, *ln_beta = nullptr;
    bf16 *ln_xhat = nullptr;
    float *ln_rstd = nullptr;
};

constexpr float kLnEps = 1e-5f;

struct DgradEpilogue {
    const bf16 *mask_act;  // [M'][Ci]: output is zeroed where this is <= 0; may be nullptr
    bf16 *out;             // [M'][Ci] bf16, or nullptr
    float *out_f32;        // [M'][Ci] fp32, or nullptr
    const uint32_t *mask_bits = nullptr;  // the same gate as one bit per element, [M'][Ci / 32] (channel c at bit gate_bit_of_channel(c) of word c / 32);
                                          // used instead of mask_act by kernels that support it
    int ksplit = 1;  // flat GEMMs with out_f32 only: the reduction is cut into ksplit (<= 4) equal slabs and slab s leaves
                     // its partial product in out_f32 + s * M' * Ci; the reader adds the slabs in order
};

// ldy: row stride (elements) of Y / dY (>= Co).  wt_ld: row stride of the innermost (co)
// dimension of the transposed weights Wt[ci][tap][wt_ld].
int tc_gemm_fwd(const ConvGeom &g, const bf16 *X, const bf16 *W, const FwdEpilogue &e, int32_t *status,
                cudaStream_t st);
int tc_gemm_dgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *Wt, int wt_ld, const DgradEpilogue &e,
                  int32_t *status, cudaStream_t st);
int tc_gemm_wgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW, float *part, size_t part_elems,
                  int32_t *status, cudaStream_t st);

// TMA-fed versions of the same three operations (operand tiles moved by cp.async.bulk.tensor).  They cover
// channel counts that are multiples of 32 (any multiple of 8 that is at least 64 for a fully connected layer);
// for anything else they return PPO_ERR_UNSUPPORTED without launching and the caller uses the tc_ versions.
int tma_gemm_fwd(const ConvGeom &g, const bf16 *X, const bf16 *W, const FwdEpilogue &e, int32_t *status,
                 cudaStream_t st);
// Wc: the layer's weights regrouped by tma_dgrad_weights for the merged four-class dgrad (convolutions only;
// fully connected layers read Wt).
int tma_gemm_dgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *Wt, int wt_ld, const bf16 *Wc,
                   const DgradEpilogue &e, int32_t *status, cudaStream_t st);
size_t tma_dgrad_weight_elems(int Ci, int k, int wt_ld);
int tma_dgrad_weights(const bf16 *W, bf16 *Wc, int Co, int k, int Ci, int wt_ld, cudaStream_t st);
// db (may be null; convolutions only): the bias gradient db[co] += sum over pixels of dY[.][co], taken from a
// column of ones beside the tap columns of X.
// Both weight-gradient GEMMs split the pixel range over CTAs; every CTA leaves its partial 128 x BN tile in `part`
// (part_elems floats of scratch, wgrad_scratch_elems(g) lets the split go as far as it wants) and wgrad_reduce adds the
// tiles to dW (and db) in split order: bit-identical results run to run.
int tma_gemm_wgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW, float *db, float *part,
                   size_t part_elems, int32_t *status, cudaStream_t st);
size_t wgrad_scratch_elems(const ConvGeom &g);
int wgrad_reduce(const float *part, int jtiles, int ctiles, int splits, int BN, int Kfwd, int Co, float *dW, float *db,
                 int ones_row, cudaStream_t st);

// bits[m][c / 32] bit (c % 32) = act[m][c] > 0, for C a multiple of 32.
int relu_bits(const bf16 *act, uint32_t *bits, long long M, int C, cudaStream_t st);

// First convolution (C_in = 1) as a tensor-core GEMM over thread-built im2col tiles (conv1_tc.cu).
// ln_* as in FwdEpilogue (all null: no normalisation); with them C1 must be 16 or 32.
int conv1_tc_fwd(const __half *depth, const bf16 *W, const float *bias, bf16 *out, uint32_t *bits, int rows, int Hi,
                 int Wi, int Ho, int Wo, int C1, int ks, const float *ln_gamma, const float *ln_beta, bf16 *ln_xhat,
                 float *ln_rstd, int32_t *status, cudaStream_t st);
