// Shared declarations of the CUDA library: status codes, handles, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/ppo_b200.h"

typedef __nv_bfloat16 bf16;

#define PPO_CUDA_CHECK(expr)                    \
    do {                                        \
        cudaError_t _e = (expr);                \
        if (_e != cudaSuccess) return PPO_ERR_CUDA; \
    } while (0)

// After every kernel launch: counts it (ppo_launch_count) and turns a launch error into a status.
#define PPO_LAUNCH_CHECK()                  \
    do {                                    \
        ppo_count_launches(1);              \
        PPO_CUDA_CHECK(cudaGetLastError()); \
    } while (0)

static inline bool ppo_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
static inline size_t ppo_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int ppo_cdiv(long long a, long long b) { return (int)((a + b - 1) / b); }

// Device status word shared by all kernels (first error wins); lives in buffer.cu.
int32_t *ppo_device_status_ptr();
// Adds n to the process-wide count of kernels and memsets this library has enqueued.
void ppo_count_launches(int n);
int ppo_num_sms();

struct ppo_buffer {
    ppo_buffer_desc d;
    char *base;
    size_t bytes;
    size_t field_off[PPO_NUM_FIELDS];
    bool gae_valid;
    int gae_blocks;  // partial sums held in the scratch slab
    bool barrier_zeroed;  // the grid-barrier words at the end of the scratch slab have been cleared once
};

// Geometry of one stride-2 convolution (an FC layer is the 1x1 image, k = 1 case).
struct ConvGeom {
    int B, Hi, Wi, Ci, Ho, Wo, Co, k, pad;
    __host__ __device__ int taps() const { return k * k; }
    __host__ __device__ long long M() const { return (long long)B * Ho * Wo; }
    __host__ __device__ int K() const { return k * k * Ci; }
};

struct ppo_tensor {
    int64_t off, size;
};

struct ppo_model {
    ppo_model_desc d;
    int L, F;
    int Hs[PPO_MAX_CONV + 1], Ws[PPO_MAX_CONV + 1], Cs[PPO_MAX_CONV + 1];  // index 0 = input image
    int hw[PPO_MAX_FC + 1];                                                // widths of h_0..h_F
    std::vector<ppo_tensor> tensors;
    // tensor index of the weight matrix of conv layer l (1..L; bias at +1, with norm gamma at +2 and beta at +3),
    // of the embedding (-1 without one) and of FC layer l (1..F; F + 1 is the head); log-sigma is the last tensor
    int ti_conv[PPO_MAX_CONV + 1], ti_embed, ti_fc[PPO_MAX_FC + 2];
    int ti_lstm[PPO_MAX_LSTM];     // W_x of LSTM layer l (W_h at +1, b at +2)
    int fc_in_w;                   // width of the first FC layer's input: hw[0], or lstm_h behind a recurrent trunk
    // recurrent trunk: the sequence the next forward/backward work on, and the workspace carve
    int seq_T, seq_Be;
    const uint8_t *seq_done;
    const float *seq_h_init, *seq_c_init;
    bf16 *lstm_hs[PPO_MAX_LSTM];     // outputs h [mb][H]
    bf16 *lstm_hprev[PPO_MAX_LSTM];  // state each step started from (after done-resets) [mb][H]
    float *lstm_c[PPO_MAX_LSTM];     // cell states [mb][H], followed by c_prev [mb][H]
    float *lstm_gates[PPO_MAX_LSTM]; // gate activations i, f, g, o [mb][4H]
    float *lstm_xg, *lstm_hg;        // W_x x of all rows [mb][4H]; W_h h_prev of one step [mb][4H]
    bf16 *lstm_dg;                   // gradient w.r.t. the gate pre-activations [mb][4H]
    float *lstm_dtop;                // gradient w.r.t. a layer's outputs [mb][H] (from the FC layers or the layer above)
    float *lstm_dhc, *lstm_dcc;      // gradients carried to the previous step [mb][H]
    size_t arena, nparams;
    // bound arrays
    float *master, *grad, *adam_m, *adam_v;
    bf16 *shadow;
    char *ws;
    size_t ws_bytes;
    int mbmax;
    // workspace carve
    bf16 *act[PPO_MAX_CONV + 1];   // act[l], l >= 1: [mb][Ho][Wo][C] post-ReLU
    bf16 *dact[PPO_MAX_CONV + 1];  // gradient w.r.t. the pre-activation of act[l]
    uint32_t *abits[PPO_MAX_CONV + 1];  // ReLU gate of act[l], one bit per element (layers with C % 32 == 0, else null)
    bf16 *xhat[PPO_MAX_CONV + 1];   // with norm: normalised values of conv layer l, [mb][Ho][Wo][C]
    float *rstd[PPO_MAX_CONV + 1];  // with norm: 1 / sqrt(var + eps) per pixel, [mb][Ho][Wo]
    bf16 *dze;                      // with embed: gradient w.r.t. the embedding's pre-activation, [mb][E]
    float *ln_part;                 // with norm: per-block partial sums of the gamma / beta gradients
    size_t ln_cap;
    bf16 *h[PPO_MAX_FC + 1];       // h[0] = [pooled, proprio]; h[l] post-ReLU
    bf16 *dh[PPO_MAX_FC + 2];      // dh[l]: gradient w.r.t. pre-activation of h[l]; dh[F+1]: head dout padded to 16
    float *dh0_f32;                // gradient w.r.t. h[0] (pooled part feeds the un-pool)
    bf16 *wT;                      // transposed bf16 weights Wt[ci][tap][co padded to 8] for the dgrad GEMMs
    int64_t wT_off[PPO_MAX_TENSORS];  // per tensor index (matrices only)
    size_t wT_elems;
    bf16 *wC;                      // conv weights regrouped for the merged dgrad: Wc[class*Ci+ci][shift][co]
    int64_t wC_off[PPO_MAX_CONV + 1];  // per conv layer l (2..L)
    size_t wC_elems;
    // scratch of the two-stage (reproducible) gradient reductions, per weight-matrix tensor index
    float *wg_part[PPO_MAX_TENSORS];  // partial tiles of the split-K weight-gradient GEMMs
    size_t wg_cap[PPO_MAX_TENSORS];   // floats
    float *cs_part[PPO_MAX_TENSORS];  // per-block partial column sums (bias gradients)
    float *c1_part;                                         // per-block partial sums of the first layer's gradients
    size_t c1_cap;
    float *loss_partials;
    float *act_mean;               // [mb][A]: Gaussian mean of ppo_policy_act before sampling
    int loss_partial_blocks;
    bool wT_valid;
    // forward/backward pairing
    int last_row0, last_rows;
    bool fwd_valid;
    // second stream of the backward pass with its fork and join events (made on first use)
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
};

__device__ __forceinline__ float bf2f(bf16 x) { return __bfloat162float(x); }

__device__ __forceinline__ void ppo_report(int32_t *status, int code) { atomicCAS(status, 0, code); }

// ReLU and conversion of two fp32 values to a packed pair of bf16 (low half = a) in one instruction.
__device__ __forceinline__ uint32_t relu_pack_bf16x2(float a, float b) {
    uint32_t r;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}

// ReLU gates of a group of 32 channels as one word: channel c sits at bit (c >> 1) + 16 (c & 1), i.e. pair j of
// packed bf16 values owns bits j (its low half, channel 2j) and 16 + j (its high half, channel 2j + 1).  With the
// halves non-negative (they come out of a ReLU), half + 0x7fff carries into its top bit exactly when it is not
// zero, so a pair costs an add, a shift and a logic operation; and a pair's two gates come back out as the mask
// of its two halves with a shift, an and, and a multiply.
__host__ __device__ __forceinline__ int gate_bit_of_channel(int c) { return ((c & 31) >> 1) + 16 * (c & 1); }
__device__ __forceinline__ uint32_t gate_bits_add(uint32_t gate, uint32_t pair, int j) {
    const uint32_t t = pair + 0x7FFF7FFFu;
    return gate | ((t >> (15 - j)) & (0x00010001u << j));
}
__device__ __forceinline__ uint32_t gate_pair_mask(uint32_t gate, int j) {
    return ((gate >> j) & 0x00010001u) * 0xFFFFu;
}
