/*
 * ppo_b200.h -- C ABI of libppo_b200.so: one PPO learner step over an on-device
 * rollout buffer of depth-image observations, for NVIDIA B200 (sm_100a).
 *
 * The library is the learner side of a disaggregated simulator/learner split
 * (Section III-B, Algorithm 2): it keeps the trajectory buffer D of one horizon
 * on the learner GPU (D <- {} ; D <- D U {(obs, actions, rew, done)}) and runs
 * TrainPPO(pi, D) on it.
 *
 * Conventions
 *  - Every function that can fail returns an int status (PPO_OK == 0).  Argument
 *    and state errors are found on the host and nothing is launched.  No function
 *    throws, exits or traps the device.
 *  - "dev" pointers are CUDA device pointers owned by the caller.  The library
 *    never allocates or frees device memory; size queries say how much the caller
 *    must provide.  *_create / *_alloc allocate only small host-side handles.
 *  - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on it and
 *    do not synchronise (ppo_poll_status is the exception).
 *  - Device pointers must be 16-byte aligned; storage handed to ppo_buffer_alloc
 *    and ppo_model_bind's workspace must be 256-byte aligned.
 *  - Samples of the buffer are numbered time-major: s = t * N + n.
 *  - Not thread-safe per handle; different handles may be used from different threads.
 */
#ifndef PPO_B200_H
#define PPO_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    PPO_OK = 0,
    PPO_ERR_INVALID_ARG = 1, /* NULL pointer, value out of range */
    PPO_ERR_SHAPE = 2,       /* sizes inconsistent with the descriptor */
    PPO_ERR_ALIGN = 3,       /* pointer not aligned as required */
    PPO_ERR_STATE = 4,       /* call out of order (e.g. gather before GAE) */
    PPO_ERR_CUDA = 5,        /* a CUDA runtime call failed */
    PPO_ERR_TIMEOUT = 6,     /* a bounded device-side wait gave up */
    PPO_ERR_UNSUPPORTED = 7  /* shape outside what the kernels implement */
};

const char *ppo_status_string(int status);

/* ------------------------------------------------------------------ buffer -- */

/* Shape of the trajectory buffer D (Algorithm 2): N envs, horizon T, depth frames
 * H x W (fp16), P proprioceptive floats and A action floats per env-step. */
typedef struct {
    int32_t N, T, H, W, P, A;
} ppo_buffer_desc;

typedef struct ppo_buffer ppo_buffer;

/* Slabs of the buffer, each time-major [T][N][...] and 256-byte aligned. */
enum {
    PPO_FIELD_DEPTH = 0,  /* fp16  [T][N][H][W] */
    PPO_FIELD_PROPRIO,    /* fp32  [T][N][P]    */
    PPO_FIELD_ACTION,     /* fp32  [T][N][A]    */
    PPO_FIELD_LOGP,       /* fp32  [T][N]  log-prob of the action under the rollout policy */
    PPO_FIELD_VALUE,      /* fp32  [T][N]  value estimate at rollout time */
    PPO_FIELD_REWARD,     /* fp32  [T][N]  */
    PPO_FIELD_DONE,       /* uint8 [T][N]  returned by the same env step as the reward */
    PPO_FIELD_ADV,        /* fp32  [T][N]  written by ppo_compute_gae */
    PPO_FIELD_RET,        /* fp32  [T][N]  written by ppo_compute_gae */
    PPO_FIELD_SCRATCH,    /* internal reduction scratch */
    PPO_NUM_FIELDS
};

/* Bytes of one slab (unpadded) for a depth element of `depth_elem_bytes` (the kernels
 * use 2; 4 reproduces the fp32 sizing example of Section III-B: 512 envs x 320x240 x
 * 16 steps = 2.5 GB).  Returns 0 for a bad descriptor or field. */
size_t ppo_buffer_field_bytes(const ppo_buffer_desc *desc, int field, int depth_elem_bytes);

/* Total device bytes ppo_buffer_alloc needs (fp16 depth, every slab padded to 256 B).
 * Returns 0 for a bad descriptor. */
size_t ppo_buffer_bytes(const ppo_buffer_desc *desc);

/* D <- {} (Algorithm 2): carves the slabs out of caller-owned device storage of at
 * least ppo_buffer_bytes(desc) bytes, 256-byte aligned.  The storage must outlive the
 * handle.  Nothing is written to the device. */
int ppo_buffer_alloc(const ppo_buffer_desc *desc, void *dev_storage, size_t bytes, ppo_buffer **out);

/* Frees the host handle only. */
int ppo_buffer_free(ppo_buffer *buf);

/* Device address of a slab (NULL on error); for callers that fill or read slabs directly. */
void *ppo_buffer_field_ptr(const ppo_buffer *buf, int field);

/* D <- D U {(obs, actions, rew, done)} for step t in [0, T) (Algorithm 2): copies one
 * step of all N envs from caller device arrays into slab row t.
 *   depth_f16 [N][H][W] fp16, proprio [N][P], action [N][A], logp [N], value [N],
 *   reward [N] (fp32), done [N] uint8.
 * Invalidates advantages computed earlier.  Errors: t outside [0,T) -> INVALID_ARG. */
int ppo_buffer_write_step(ppo_buffer *buf, int t, const void *dev_depth_f16, const float *dev_proprio,
                          const float *dev_action, const float *dev_logp, const float *dev_value,
                          const float *dev_reward, const uint8_t *dev_done, void *stream);

/* The two halves of the same insertion for a rollout whose actions come from ppo_policy_act (Algorithm 2:
 * obs arrives, actions <- pi(obs), the env step returns rew and done): ppo_buffer_write_obs copies the
 * observation of step t (depth_f16 [N][H][W] fp16, proprio [N][P]) into slab row t before the policy runs,
 * ppo_buffer_write_outcome the reward [N] fp32 and done [N] uint8 afterwards; action, log-prob and value of
 * row t are written in place by ppo_policy_act.  Same errors and invalidation as ppo_buffer_write_step. */
int ppo_buffer_write_obs(ppo_buffer *buf, int t, const void *dev_depth_f16, const float *dev_proprio, void *stream);
int ppo_buffer_write_outcome(ppo_buffer *buf, int t, const float *dev_reward, const uint8_t *dev_done, void *stream);

/* Synthetic depth producer, standing in for the simulator's depth rendering (Section III-C; Algorithm 1 renders,
 * Algorithm 2 receives): ray-casts one small analytic scene per env straight into the DEPTH slab at row t, as fp16.
 * Pinhole camera at the origin looking along +z with horizontal field of view hfov (radians); pixel (v, u) sees the
 * ray through ((u + 0.5 - W/2) / f, (v + 0.5 - H/2) / f, 1), f = (W/2) / tan(hfov/2).  The scene of env n is the
 * plane normal . p = offset (dev_plane [N][4] = {nx, ny, nz, offset}, unit normal) and n_prims (<= 32) primitives,
 * dev_prims [N][n_prims][8] = {type, x, y, z, p0, p1, p2, p3}: type 0 sphere (centre, radius p0), 1 axis-aligned box
 * (centre, half extents p0..p2), 2 capsule (segment from (x,y,z) to (x,y,z) + (p0,p1,p2), radius p3).  A pixel gets
 * the z coordinate of the nearest hit if it lies in [near, far], else 0 (no return).  fp32 arithmetic.
 * Invalidates advantages computed earlier.  Errors: t outside [0,T), n_prims outside [0,32], bad camera values ->
 * INVALID_ARG. */
int ppo_buffer_render_depth(ppo_buffer *buf, int t, float hfov, float near, float far, const float *dev_plane,
                            int n_prims, const float *dev_prims, void *stream);

/* First stage of TrainPPO (Algorithm 2): generalised advantage estimation per env by a
 * reverse scan over t,
 *   delta_t = r_t + gamma V_{t+1} (1 - d_t) - V_t,  A_t = delta_t + gamma lambda (1 - d_t) A_{t+1},
 *   R_t = A_t + V_t,  V_T = dev_last_value[n],  A_T = 0,
 * written to the ADV and RET slabs; then, if normalize != 0, the advantages of the whole
 * buffer are replaced by (A - mean) / (std + 1e-8) with the unbiased (M-1) standard
 * deviation.  dev_stats_out (may be NULL) receives {mean, std} of the raw advantages as
 * fp32 when normalize != 0.  fp32 arithmetic, fp64 accumulation of the moments.
 * normalize == 1 runs the scan and the normalisation as two launches; normalize == 2 runs both as one cooperative
 * launch with a bounded grid barrier in between (the same arithmetic; the fp64 partial moments of more than 32 blocks
 * are added in a different fixed order, which the rounding of mean and deviation to fp32 all but always hides;
 * PPO_ERR_UNSUPPORTED when the scan's blocks, one per 128 envs, cannot all be resident at once). */
int ppo_compute_gae(ppo_buffer *buf, const float *dev_last_value, float gamma, float lambda, int normalize,
                    float *dev_stats_out, void *stream);

/* No counterpart in the paper: a convenience for callers that are not allowed to allocate device
 * memory.  Some users of this library run it from places where cudaMalloc is off limits: inside a
 * host process that hands out one fixed arena and forbids further allocations, under a memory
 * budget that is fixed before the learner starts, or from code that must not synchronise the
 * device (cudaMalloc and cudaFree may).  ppo_compute_gae needs a small scratch area for the partial
 * sums of the advantage moments, which normally comes out of the buffer storage that the caller
 * allocated for ppo_buffer_alloc.  This variant works on bare arrays and keeps that scratch in a
 * fixed array inside the library image instead, so it never allocates and never frees: no
 * cudaMalloc, cudaFree or allocating library routine is called, here or by anything it calls.
 *
 * Same arithmetic as ppo_compute_gae, on caller-owned device arrays (time-major, s = t*N + n):
 *   in : dev_reward, dev_value fp32 [T][N]; dev_done uint8 [T][N]; dev_last_value fp32 [N]
 *   out: dev_adv, dev_ret fp32 [T][N] (dev_adv 16-byte aligned); dev_stats_out fp32 [2] = {mean, std}
 *        of the raw advantages when normalize != 0 (may be NULL).
 * Limits and caveats:
 *  - at most PPO_GAE_STATIC_MAX_ENVS envs (N); more returns PPO_ERR_UNSUPPORTED and launches nothing.
 *    The scratch is 64 KiB and every GPU that loads the library holds it until the process exits.
 *  - the first call on each device looks up the scratch array's device address (with that device
 *    current); make that first call outside any stream capture.  If the library's code has not been
 *    loaded onto the device yet, that first call also makes the CUDA runtime load it, which may
 *    allocate and synchronise inside the driver; later calls do neither.
 *  - all calls on a device share the one scratch array, and it keeps whatever the last call left in
 *    it.  Each call overwrites every entry it later reads, so nothing needs clearing, but two calls
 *    whose kernels can overlap on the GPU (different streams, no dependency) race on it: serialise them.
 * Errors: NULL pointers, T or N <= 0, gamma or lambda outside [0, 1] -> PPO_ERR_INVALID_ARG;
 * misaligned dev_adv -> PPO_ERR_ALIGN; failure to find the scratch address -> PPO_ERR_CUDA. */
#define PPO_GAE_STATIC_MAX_ENVS 524288
int ppo_gae_static(const float *dev_reward, const float *dev_value, const uint8_t *dev_done,
                   const float *dev_last_value, int T, int N, float gamma, float lambda, int normalize,
                   float *dev_adv, float *dev_ret, float *dev_stats_out, void *stream);

/* One gathered minibatch: caller-allocated device arrays of B rows. */
typedef struct {
    void *depth_f16;  /* [B][H][W] fp16 */
    float *proprio;   /* [B][P] */
    float *action;    /* [B][A] */
    float *logp_old;  /* [B] */
    float *value_old; /* [B] */
    float *adv;       /* [B] */
    float *ret;       /* [B] */
    uint32_t *index;  /* [B] sample numbers s of the rows; may be NULL */
    int32_t B;
} ppo_minibatch;

/* Minibatch mb_index of num_minibatches for (seed, epoch): row j receives an exact copy
 * of sample s = pi(mb_index * B + j), where pi is the seeded bijection on [0, M), M = N*T:
 * a 6-round balanced Feistel network on 2h bits, h = max(1, ceil(ceil_log2(M) / 2)), with
 * cycle walking; round function mix32(R ^ key_j) & (2^h - 1); all arithmetic uint32.
 *   mix32(x): x ^= x>>16; x *= 0x9E3779B9; x ^= x>>15; x *= 0x6A09E667; x ^= x>>16
 *   key_j = mix32(lo32(seed) ^ mix32(hi32(seed) + 0x9E3779B9*(j+1)) ^ mix32(epoch + 0xBB67AE85*(j+1)))
 * Requires M % num_minibatches == 0 and out->B == M / num_minibatches (else SHAPE), and
 * a prior ppo_compute_gae since the last write_step (else STATE). */
int ppo_shuffle_gather_minibatch(const ppo_buffer *buf, uint64_t seed, uint32_t epoch, int mb_index,
                                 int num_minibatches, const ppo_minibatch *out, void *stream);

/* ------------------------------------------------------------------- model -- */

#define PPO_MAX_CONV 8
#define PPO_MAX_FC 4
#define PPO_MAX_LSTM 4
#define PPO_MAX_TENSORS (4 * PPO_MAX_CONV + 2 * PPO_MAX_FC + 3 * PPO_MAX_LSTM + 5)

/* Policy/value network (Section III-C: CNN with ReLU on the depth image, joined with
 * proprioception, fully connected layers).  Conv l: k x k cross-correlation, stride 2,
 * zero padding k/2, ReLU; global average pool; concat [pooled, proprio]; hidden FC layers
 * with ReLU; one linear head giving the Gaussian mean (A) and the value (1); log-sigma is a
 * free A-vector.  Channel counts of conv layers >= 1 and FC widths must be multiples of 8.
 *
 * The depth CNN as Section III-C words it ("4-layer CNN ... layer normalization, and ReLU", "a fully connected
 * layer which outputs a 32 dimensional embedding for the depth") is selected by the last two fields, both 0 for
 * the plain network above:
 *   norm != 0 : every conv output is layer-normalised over its channels at each pixel before the ReLU,
 *               y = ReLU(gamma * (z - mean) / sqrt(var + 1e-5) + beta), mean and (biased) variance over the C
 *               channels of the pixel, gamma and beta learned per channel.  Needs conv_c[0] in {16, 32}, every
 *               conv_c <= 256 and an even frame width.
 *   embed > 0 : instead of the global average pool, the last conv output is flattened (pixel-major, channel
 *               innermost) and mapped by a fully connected layer with ReLU to `embed` values (a multiple of 32,
 *               embed + P a multiple of 8), which are concatenated with proprio.
 *
 * The recurrent trunk of Section III-C ("two LSTM layers with 1024 units" between that joined feature and the fully
 * connected layers) is selected by n_lstm > 0 (up to 4 layers of lstm_h units, lstm_h a multiple of 64):
 *   (i, f, g, o) = (sigmoid, sigmoid, tanh, sigmoid)(W_x x_t + W_h h_prev + b),  c_t = f c_prev + i g,  h_t = o tanh(c_t)
 * per layer and time step.  Such a model works on sequence minibatches (ppo_shuffle_gather_sequences) whose rows are
 * time-major, row = t * Be + e, announced with ppo_model_set_sequence; ppo_encoder_fwd / ppo_encoder_bwd then take
 * the whole minibatch (rows == T * Be), the backward pass being back-propagation through the T steps. */
typedef struct {
    int32_t H, W;
    int32_t n_conv;
    int32_t conv_c[PPO_MAX_CONV];
    int32_t conv_k[PPO_MAX_CONV];
    int32_t n_fc;
    int32_t fc[PPO_MAX_FC];
    int32_t P, A;
    int32_t norm, embed;
    int32_t n_lstm, lstm_h;
} ppo_model_desc;

typedef struct ppo_model ppo_model;

int ppo_model_create(const ppo_model_desc *desc, ppo_model **out);
int ppo_model_destroy(ppo_model *m);

/* Parameter vector ("arena") layout: tensors in the order conv W_l [Cout][k][k][Cin],
 * conv b_l [Cout] (with norm: followed by gamma_l [Cout], beta_l [Cout]), ..., (with embed: embed W
 * [E][Ho*Wo*C_L], embed b [E],) (per LSTM layer: W_x [4H][in], W_h [4H][H], b [4H], gate blocks in the order input,
 * forget, cell, output,) fc W [out][in], fc b [out], ..., head W [A+1][hid] (rows 0..A-1
 * mean, row A value), head b [A+1], log-sigma [A]; every tensor starts at a multiple of 64
 * elements; gaps are zero and stay zero.  The same offsets index master, shadow, gradient
 * and Adam moment arrays. */
size_t ppo_model_param_count(const ppo_model *m); /* sum of tensor sizes, without gaps */
size_t ppo_model_arena_elems(const ppo_model *m); /* length of the arrays, with gaps */
int ppo_model_num_tensors(const ppo_model *m);
int ppo_model_tensor_info(const ppo_model *m, int index, int64_t *offset, int64_t *size);

/* Device bytes of workspace for forward+backward of up to `microbatch` rows at a time. */
size_t ppo_model_workspace_bytes(const ppo_model *m, int microbatch);

/* Attaches caller-owned device arrays: master/grad/adam_m/adam_v fp32 [arena_elems],
 * shadow_bf16 bf16 [arena_elems] (weights as the GEMMs read them; refreshed by
 * ppo_adam_step and ppo_model_sync_shadow), workspace of ws_bytes >=
 * ppo_model_workspace_bytes(m, microbatch). */
int ppo_model_bind(ppo_model *m, float *dev_master, void *dev_shadow_bf16, float *dev_grad, float *dev_adam_m,
                   float *dev_adam_v, void *dev_workspace, size_t ws_bytes, int microbatch);

/* Describes the sequence minibatch the next ppo_encoder_fwd / ppo_encoder_bwd of a recurrent model work on: T time
 * steps of Be envs, rows time-major; dev_done uint8 [T][Be] (the flags stored with the steps: a set flag zeroes the
 * state the NEXT step starts from); dev_h_init, dev_c_init fp32 [n_lstm][Be][lstm_h], the state the first step starts
 * from (constants of the backward pass).  The pointers are read by those calls, not copied.  T * Be must not
 * exceed the bound micro-batch.  Errors: model without LSTM layers -> STATE; bad sizes -> SHAPE. */
int ppo_model_set_sequence(ppo_model *m, int T, int Be, const uint8_t *dev_done, const float *dev_h_init,
                           const float *dev_c_init);

/* The recurrent state the step AFTER the announced sequence starts from (Algorithm 2 keeps acting with the policy from
 * one buffer fill to the next): dev_h_out, dev_c_out fp32 [n_lstm][Be][lstm_h] receive h and c of the last time step of
 * the latest ppo_encoder_fwd (h as the layers pass it on, i.e. rounded to bf16), zeroed where that step's done flag is
 * set.  They may be the arrays a later ppo_model_set_sequence names as the initial state, but not the ones the
 * current sequence was announced with while its backward pass is still to run.  Errors: no forward since the sequence
 * was announced, or a model without LSTM layers -> STATE. */
int ppo_model_read_state(const ppo_model *m, float *dev_h_out, float *dev_c_out, void *stream);

/* shadow <- bf16(master) (round to nearest even); call after writing master from outside. */
int ppo_model_sync_shadow(ppo_model *m, void *stream);

/* Forward of rows [row0, row0+rows) of a minibatch (rows <= bound microbatch): writes the
 * Gaussian mean dev_mean [rows][A] and the value dev_value [rows] (fp32) and keeps the
 * activations in the workspace for ppo_encoder_bwd.  bf16 operands (weights from the
 * shadow, activations rounded to bf16 between layers), fp32 accumulation; the depth
 * frame enters as fp16. */
int ppo_encoder_fwd(ppo_model *m, const ppo_minibatch *mb, int row0, int rows, float *dev_mean, float *dev_value,
                    void *stream);

/* PPO-clip loss of rows [row0, row0+rows) fused with its gradient (TrainPPO, Algorithm 2):
 *   z = (a - mu)/sigma, sigma = exp(logsigma);  logp = sum_j [-z_j^2/2 - logsigma_j - ln(2 pi)/2]
 *   r = exp(logp - logp_old);  s = min(r Adv, clamp(r, 1-clip, 1+clip) Adv)
 *   L = -mean(s) + vf_coef mean((V - R)^2) - ent_coef H,  H = sum_j logsigma_j + (A/2)(1 + ln 2 pi)
 * with means over B_total rows (so micro-batches add up to the minibatch).  Writes
 * dL/dmu to dev_dmean [rows][A] and dL/dV to dev_dvalue [rows]; ADDS dL/dlogsigma into the
 * log-sigma slot of the bound gradient array and ADDS this call's share of
 * {L_pi, L_V, H, approx_kl = mean(logp_old - logp), clip_fraction} into dev_loss_out[5]
 * (the caller zeroes both at the start of a minibatch).  At a tie of the min the unclipped
 * branch is taken. */
int ppo_loss_fwd_bwd(ppo_model *m, const ppo_minibatch *mb, int row0, int rows, int B_total, const float *dev_mean,
                     const float *dev_value, float clip, float vf_coef, float ent_coef, float *dev_loss_out,
                     float *dev_dmean, float *dev_dvalue, void *stream);

/* Backward of the rows of the latest ppo_encoder_fwd (same row0/rows, else STATE): adds
 * (accumulate != 0) or writes (accumulate == 0, the log-sigma slot is left as it is)
 * dL/dtheta into the bound gradient array, with respect to the fp32 master (straight
 * through the bf16 rounding).  Weight-gradient kernels that do not feed the chain of
 * input gradients run on a second stream the model creates at its first backward pass;
 * that stream forks from `stream` and has joined it again when the call returns, so the
 * caller sees the ordering of a single stream. */
int ppo_encoder_bwd(ppo_model *m, const ppo_minibatch *mb, int row0, int rows, const float *dev_dmean,
                    const float *dev_dvalue, int accumulate, void *stream);

/* Where the forward keeps what the backward reads (inside the bound workspace): kind 0 =
 * conv activation of layer `index` in 1..n_conv, NHWC bf16 [rows][Ho][Wo][C]; kind 1 = h_index
 * for index in 0..n_fc, bf16 [rows][width] (h_0 = [pooled, proprio]); kind 2 = the ReLU gate bits of conv
 * activation `index` (only for layers below the last whose channel count is a multiple of 32, else INVALID_ARG),
 * uint32 [rows][Ho][Wo][C/32] (kind 3 and 4, with norm only: the normalised values xhat of conv layer `index`,
 * bf16 [rows][Ho][Wo][C], and their reciprocal standard deviations, fp32 [rows][Ho][Wo]; kind 5, 6, 7, 8, with
 * LSTM layers only, index = layer 0..n_lstm-1: the layer's outputs h bf16 [rows][lstm_h], its cell states c fp32
 * [rows][lstm_h], its gate activations fp32 [rows][4 lstm_h], and the states its steps started from, h_prev bf16
 * [rows][lstm_h] (c_prev fp32 [rows][lstm_h] follows the cell states: kind 6 has 2 rows lstm_h elements)); channel c belongs to word c / 32 and sits at bit ((c % 32) / 2) + 16 * (c % 2) of it (the
 * two halves of a packed pair of bf16 values own bits j and 16 + j), set where the activation is > 0.  *elems is the capacity
 * for the bound micro-batch.  For inspection and for tests that substitute the saved
 * activations between ppo_encoder_fwd and ppo_encoder_bwd. */
int ppo_model_activation_ptr(const ppo_model *m, int kind, int index, void **dev_ptr, size_t *elems);

/* Recomputes the one-bit-per-element ReLU gates the backward pass reads from the saved conv activations of
 * the first `rows` rows.  ppo_encoder_fwd keeps them up to date itself; call this only after writing saved
 * activations from outside (see ppo_model_activation_ptr) and before ppo_encoder_bwd. */
int ppo_model_sync_masks(ppo_model *m, int rows, void *stream);

/* Zeroes the bound gradient array (start of a minibatch). */
int ppo_model_zero_grad(ppo_model *m, void *stream);

/* Adam over the whole arena in one pass (bias-corrected, eps outside the square root, no
 * weight decay), step >= 1:  m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
 * theta <- theta - lr (m/(1-b1^step)) / (sqrt(v/(1-b2^step)) + eps); shadow <- bf16(theta). */
int ppo_adam_step(ppo_model *m, float lr, float beta1, float beta2, float eps, int64_t step, void *stream);

/* Sequence minibatch mb_index of num_minibatches for (seed, epoch), for recurrent policies (Section III-C: the LSTM
 * needs every env's steps in order): the ENVS are permuted with the same seeded bijection, now on [0, N), and a
 * minibatch holds Be = N / num_minibatches envs with all their T steps, rows time-major: row t * Be + e is an exact
 * copy of sample t * N + pi(mb_index * Be + e).  out->B must be T * Be; dev_done_out uint8 [T][Be] receives the done
 * flags of the rows; out->index (optional) the sample numbers.  Requires N % num_minibatches == 0 (else SHAPE) and a
 * prior ppo_compute_gae (else STATE). */
int ppo_shuffle_gather_sequences(const ppo_buffer *buf, uint64_t seed, uint32_t epoch, int mb_index, int num_minibatches,
                                 const ppo_minibatch *out, uint8_t *dev_done_out, void *stream);

/* Rollout-time action of the policy (Algorithm 2, actions <- pi(obs)) given the mean from
 * ppo_encoder_fwd and caller-supplied standard-normal noise dev_eps [rows][A]:
 * action = mu + exp(logsigma) * eps, logp = its log-density.  Outputs fp32 [rows][A], [rows]. */
int ppo_policy_sample(const ppo_model *m, int rows, const float *dev_mean, const float *dev_eps, float *dev_action,
                      float *dev_logp, void *stream);

/* actions <- pi(stack(obs)) followed by D <- D U {...} without a copy in between (Algorithm 2): runs the
 * encoder on the observation already stored in slab row t of `buf` (all N envs, in micro-batches of the bound
 * size), draws action = mu + exp(logsigma) * eps from caller-supplied standard-normal noise dev_eps [N][A],
 * and writes the action, its log-density and the value estimate straight into the ACTION, LOGP and VALUE
 * slabs at row t (ppo_buffer_field_ptr gives the simulator the address to read the actions from).
 * Invalidates advantages computed earlier and the saved activations of the last ppo_encoder_fwd.
 * Errors: t outside [0,T) -> INVALID_ARG; buffer and model shapes (H, W, P, A) differ -> SHAPE. */
int ppo_policy_act(ppo_model *m, ppo_buffer *buf, int t, const float *dev_eps, void *stream);

/* Number of kernels and memsets the library has enqueued in this process so far (all handles, all
 * devices).  Instrumentation for benchmarks that report launches per step; no counterpart in the paper. */
uint64_t ppo_launch_count(void);

/* Self-test of the bounded waits (no counterpart in the paper): every device-side wait of the pipelined
 * kernels gives up after a cycle limit, records PPO_ERR_TIMEOUT in the status word and lets the kernel
 * return.  This launches one small kernel whose 64 threads run that same wait, with a limit of
 * limit_cycles (1 .. 2e9) clock cycles, on a barrier that nothing completes; *dev_gave_up (device int,
 * zeroed by the caller) receives the number of threads that left the wait unsatisfied.  The next
 * ppo_poll_status returns PPO_ERR_TIMEOUT and clears it; the device stays usable. */
int ppo_selftest_wait_timeout(long long limit_cycles, int *dev_gave_up, void *stream);

/* Synchronises `stream`, then returns the first error a kernel recorded in the library's
 * device status word since the last poll (PPO_OK if none), or PPO_ERR_CUDA if the stream
 * reports a CUDA error. */
int ppo_poll_status(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PPO_B200_H */
