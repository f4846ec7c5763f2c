// Model handle (parameter arena layout, workspace carve), fused PPO loss + gradient,
// Gaussian action sampling and the fused Adam pass.
#include <math.h>

#include <new>

#include "common.cuh"
#include "gemm.cuh"

static int conv_out(int in, int k) { return (in + 2 * (k / 2) - k) / 2 + 1; }

extern "C" int ppo_model_create(const ppo_model_desc *d, ppo_model **out) {
    if (!out) return PPO_ERR_INVALID_ARG;
    *out = nullptr;
    if (!d) return PPO_ERR_INVALID_ARG;
    if (d->H <= 0 || d->W <= 0 || d->n_conv < 1 || d->n_conv > PPO_MAX_CONV || d->n_fc < 0 || d->n_fc > PPO_MAX_FC ||
        d->P <= 0 || d->A <= 0 || d->A > 15)
        return PPO_ERR_INVALID_ARG;
    for (int l = 0; l < d->n_conv; ++l) {
        if (d->conv_c[l] <= 0 || d->conv_c[l] % 8 != 0 || d->conv_c[l] > 512) return PPO_ERR_UNSUPPORTED;
        if (d->conv_k[l] < 1 || d->conv_k[l] % 2 == 0 || d->conv_k[l] > 7) return PPO_ERR_UNSUPPORTED;
    }
    if (d->conv_c[0] > 64) return PPO_ERR_UNSUPPORTED;  // first layer runs as a direct convolution
    if (d->conv_c[0] * (d->conv_k[0] * d->conv_k[0] + 1) > 2048) return PPO_ERR_UNSUPPORTED;
    for (int l = 0; l < d->n_fc; ++l)
        if (d->fc[l] <= 0 || d->fc[l] % 8 != 0) return PPO_ERR_UNSUPPORTED;
    if (d->embed < 0) return PPO_ERR_INVALID_ARG;
    if (d->embed > 0 && (d->embed % 32 != 0 || (d->embed + d->P) % 8 != 0 || d->embed > 256)) return PPO_ERR_UNSUPPORTED;
    if (d->embed == 0 && (d->conv_c[d->n_conv - 1] + d->P) % 8 != 0) return PPO_ERR_UNSUPPORTED;
    if (d->norm) {
        // the normalisation runs in the forward kernels' epilogues, where one thread owns all channels of a pixel
        if ((d->conv_c[0] != 16 && d->conv_c[0] != 32) || d->W % 2 != 0 || d->conv_k[0] == 1) return PPO_ERR_UNSUPPORTED;
        for (int l = 0; l < d->n_conv; ++l)  // 16, 32, 64, 128 or 256 channels: a pixel's channels split evenly over lanes
            if (d->conv_c[l] > 256 || d->conv_c[l] < 16 || (d->conv_c[l] & (d->conv_c[l] - 1)) != 0) return PPO_ERR_UNSUPPORTED;
    }
    if (d->n_lstm < 0 || d->n_lstm > PPO_MAX_LSTM) return PPO_ERR_INVALID_ARG;
    if (d->n_lstm > 0 && (d->lstm_h <= 0 || d->lstm_h % 64 != 0 || d->lstm_h > 4096)) return PPO_ERR_UNSUPPORTED;
    if (d->n_lstm > 0 && ((d->embed > 0 ? d->embed : d->conv_c[d->n_conv - 1]) + d->P) % 64 != 0)
        return PPO_ERR_UNSUPPORTED;  // the trunk's input rows feed 64-channel boxes
    ppo_model *m = new (std::nothrow) ppo_model();
    if (!m) return PPO_ERR_INVALID_ARG;
    m->d = *d;
    m->L = d->n_conv;
    m->F = d->n_fc;
    m->Hs[0] = d->H;
    m->Ws[0] = d->W;
    m->Cs[0] = 1;
    for (int l = 0; l < m->L; ++l) {
        m->Hs[l + 1] = conv_out(m->Hs[l], d->conv_k[l]);
        m->Ws[l + 1] = conv_out(m->Ws[l], d->conv_k[l]);
        m->Cs[l + 1] = d->conv_c[l];
    }
    m->hw[0] = (d->embed > 0 ? d->embed : m->Cs[m->L]) + d->P;
    for (int l = 0; l < m->F; ++l) m->hw[l + 1] = d->fc[l];
    int64_t off = 0;
    size_t count = 0;
    auto push = [&](int64_t sz) {
        m->tensors.push_back({off, sz});
        off += (sz + 63) / 64 * 64;
        count += (size_t)sz;
    };
    for (int l = 0; l < m->L; ++l) {
        m->ti_conv[l + 1] = (int)m->tensors.size();
        push((int64_t)m->Cs[l + 1] * d->conv_k[l] * d->conv_k[l] * m->Cs[l]);
        push(m->Cs[l + 1]);
        if (d->norm) {
            push(m->Cs[l + 1]);
            push(m->Cs[l + 1]);
        }
    }
    m->ti_embed = -1;
    if (d->embed > 0) {
        m->ti_embed = (int)m->tensors.size();
        push((int64_t)d->embed * m->Hs[m->L] * m->Ws[m->L] * m->Cs[m->L]);
        push(d->embed);
    }
    m->fc_in_w = m->hw[0];
    for (int l = 0; l < d->n_lstm; ++l) {
        m->ti_lstm[l] = (int)m->tensors.size();
        push((int64_t)4 * d->lstm_h * m->fc_in_w);
        push((int64_t)4 * d->lstm_h * d->lstm_h);
        push((int64_t)4 * d->lstm_h);
        m->fc_in_w = d->lstm_h;
    }
    for (int l = 0; l < m->F; ++l) {
        m->ti_fc[l + 1] = (int)m->tensors.size();
        push((int64_t)m->hw[l + 1] * (l == 0 ? m->fc_in_w : m->hw[l]));
        push(m->hw[l + 1]);
    }
    m->ti_fc[m->F + 1] = (int)m->tensors.size();
    push((int64_t)(d->A + 1) * (m->F == 0 ? m->fc_in_w : m->hw[m->F]));
    push(d->A + 1);
    push(d->A);
    m->arena = (size_t)off;
    m->nparams = count;
    {   // transposed copies of the weight matrices (conv layers >= 2, FC layers, head)
        int64_t toff = 0;
        for (size_t i = 0; i < m->tensors.size(); ++i) m->wT_off[i] = 0;
        auto tpush = [&](int ti, int64_t Ci, int64_t taps, int64_t Co) {
            m->wT_off[ti] = toff;
            toff += (Ci * taps * ((Co + 7) / 8 * 8) + 63) / 64 * 64;
        };
        for (int l = 2; l <= m->L; ++l) tpush(m->ti_conv[l], m->Cs[l - 1], d->conv_k[l - 1] * d->conv_k[l - 1], m->Cs[l]);
        if (m->ti_embed >= 0) tpush(m->ti_embed, (int64_t)m->Hs[m->L] * m->Ws[m->L] * m->Cs[m->L], 1, d->embed);
        for (int l = 0; l < d->n_lstm; ++l) {  // W_x^T [in][4H] and W_h^T [H][4H]
            tpush(m->ti_lstm[l], 4 * d->lstm_h, 1, l == 0 ? m->hw[0] : d->lstm_h);
            tpush(m->ti_lstm[l] + 1, 4 * d->lstm_h, 1, d->lstm_h);
        }
        for (int l = 1; l <= m->F + 1; ++l)
            tpush(m->ti_fc[l], l == 1 ? m->fc_in_w : m->hw[l - 1], 1, l <= m->F ? m->hw[l] : d->A + 1);
        m->wT_elems = (size_t)toff;
        int64_t coff = 0;
        for (int l = 0; l <= PPO_MAX_CONV; ++l) m->wC_off[l] = 0;
        for (int l = 2; l <= m->L; ++l) {
            m->wC_off[l] = coff;
            coff += ((int64_t)tma_dgrad_weight_elems(m->Cs[l - 1], d->conv_k[l - 1], (m->Cs[l] + 7) / 8 * 8) + 63) / 64 * 64;
        }
        m->wC_elems = (size_t)coff;
    }
    m->master = m->grad = m->adam_m = m->adam_v = nullptr;
    m->shadow = nullptr;
    m->ws = nullptr;
    m->ws_bytes = 0;
    m->mbmax = 0;
    m->fwd_valid = false;
    m->wT_valid = false;
    m->last_row0 = m->last_rows = -1;
    m->seq_T = m->seq_Be = 0;
    m->seq_done = nullptr;
    m->seq_h_init = m->seq_c_init = nullptr;
    *out = m;
    return PPO_OK;
}

extern "C" int ppo_model_destroy(ppo_model *m) {
    if (!m) return PPO_ERR_INVALID_ARG;
    if (m->side) {
        cudaStreamSynchronize(m->side);
        cudaStreamDestroy(m->side);
        cudaEventDestroy(m->ev_fork);
        cudaEventDestroy(m->ev_join);
    }
    delete m;
    return PPO_OK;
}

extern "C" size_t ppo_model_param_count(const ppo_model *m) { return m ? m->nparams : 0; }
extern "C" size_t ppo_model_arena_elems(const ppo_model *m) { return m ? m->arena : 0; }
extern "C" int ppo_model_num_tensors(const ppo_model *m) { return m ? (int)m->tensors.size() : 0; }
extern "C" int ppo_model_tensor_info(const ppo_model *m, int i, int64_t *off, int64_t *size) {
    if (!m || i < 0 || i >= (int)m->tensors.size() || !off || !size) return PPO_ERR_INVALID_ARG;
    *off = m->tensors[i].off;
    *size = m->tensors[i].size;
    return PPO_OK;
}

static const int kLossThreads = 128;

// Walks the workspace carve; with base == nullptr only sizes are computed.
static size_t carve(ppo_model *m, const ppo_model *shape, int mb, char *base) {
    size_t off = 0;
    auto take = [&](size_t bytes) -> char * {
        char *p = base ? base + off : nullptr;
        off += ppo_align_up(bytes, 256);
        return p;
    };
    for (int l = 1; l <= shape->L; ++l) {
        size_t bytes = (size_t)mb * shape->Hs[l] * shape->Ws[l] * shape->Cs[l] * sizeof(bf16);
        char *a = take(bytes), *g = take(bytes);
        if (m) { m->act[l] = (bf16 *)a; m->dact[l] = (bf16 *)g; }
        const bool bits = shape->Cs[l] % 32 == 0 && l < shape->L;  // gate bits for the dgrad of layer l + 1
        char *bt = bits ? take(bytes / 16) : nullptr;
        if (m) m->abits[l] = (uint32_t *)bt;
        char *xh = shape->d.norm ? take(bytes) : nullptr;
        char *rs = shape->d.norm ? take((size_t)mb * shape->Hs[l] * shape->Ws[l] * sizeof(float)) : nullptr;
        if (m) { m->xhat[l] = (bf16 *)xh; m->rstd[l] = (float *)rs; }
    }
    for (int l = 0; l <= shape->F; ++l) {
        size_t bytes = (size_t)mb * shape->hw[l] * sizeof(bf16);
        char *a = take(bytes), *g = take(bytes);
        if (m) { m->h[l] = (bf16 *)a; m->dh[l] = (bf16 *)g; }
    }
    {
        char *g = take((size_t)mb * 16 * sizeof(bf16));
        if (m) m->dh[shape->F + 1] = (bf16 *)g;
        char *f = take((size_t)mb * shape->hw[0] * sizeof(float));
        if (m) m->dh0_f32 = (float *)f;
        char *w = take(shape->wT_elems * sizeof(bf16));
        if (m) m->wT = (bf16 *)w;
        char *wc = take(shape->wC_elems * sizeof(bf16));
        if (m) m->wC = (bf16 *)wc;
        int blocks = ppo_cdiv(mb, kLossThreads);
        char *lp = take((size_t)blocks * 32 * sizeof(float));
        if (m) { m->loss_partials = (float *)lp; m->loss_partial_blocks = blocks; }
        char *am = take((size_t)mb * shape->d.A * sizeof(float));
        if (m) m->act_mean = (float *)am;
        // scratch of the two-stage gradient reductions (sizes do not depend on the micro-batch)
        const int sms = ppo_num_sms();
        const size_t c1 = (size_t)6 * sms * shape->Cs[1] * (shape->d.conv_k[0] * shape->d.conv_k[0] + 1);
        char *c1p = take(c1 * sizeof(float));
        if (m) { m->c1_part = (float *)c1p; m->c1_cap = c1; }
        auto scratch_for = [&](int ti, int Ci, int Co, int k) {
            ConvGeom g = {};
            g.Ci = Ci; g.Co = Co; g.k = k;
            const size_t we = wgrad_scratch_elems(g);
            char *wp = take(we * sizeof(float));
            char *cp = take((size_t)4 * sms * (Co < 16 ? 16 : Co) * sizeof(float));
            if (m) { m->wg_part[ti] = (float *)wp; m->wg_cap[ti] = we; m->cs_part[ti] = (float *)cp; }
        };
        for (int l = 2; l <= shape->L; ++l) scratch_for(shape->ti_conv[l], shape->Cs[l - 1], shape->Cs[l], shape->d.conv_k[l - 1]);
        if (shape->ti_embed >= 0)
            scratch_for(shape->ti_embed, shape->Hs[shape->L] * shape->Ws[shape->L] * shape->Cs[shape->L], shape->d.embed, 1);
        for (int l = 1; l <= shape->F + 1; ++l)
            scratch_for(shape->ti_fc[l], l == 1 ? shape->fc_in_w : shape->hw[l - 1], l <= shape->F ? shape->hw[l] : shape->d.A + 1, 1);
        if (shape->d.n_lstm > 0) {
            const size_t H = (size_t)shape->d.lstm_h, R = (size_t)mb;
            for (int l = 0; l < shape->d.n_lstm; ++l) {
                scratch_for(shape->ti_lstm[l], l == 0 ? shape->hw[0] : (int)H, 4 * (int)H, 1);
                scratch_for(shape->ti_lstm[l] + 1, (int)H, 4 * (int)H, 1);
                char *a = take(R * H * sizeof(bf16)), *b = take(R * H * sizeof(bf16));
                char *c = take(2 * R * H * sizeof(float)), *g = take(4 * R * H * sizeof(float));
                if (m) {
                    m->lstm_hs[l] = (bf16 *)a; m->lstm_hprev[l] = (bf16 *)b;
                    m->lstm_c[l] = (float *)c; m->lstm_gates[l] = (float *)g;
                }
            }
            char *xg = take(4 * R * H * sizeof(float)), *hg = take(4 * R * H * sizeof(float));
            char *dg = take(4 * R * H * sizeof(bf16)), *dt = take(R * H * sizeof(float));
            char *dh = take(R * H * sizeof(float)), *dc = take(R * H * sizeof(float));
            if (m) {
                m->lstm_xg = (float *)xg; m->lstm_hg = (float *)hg; m->lstm_dg = (bf16 *)dg;
                m->lstm_dtop = (float *)dt; m->lstm_dhc = (float *)dh; m->lstm_dcc = (float *)dc;
            }
        }
        if (shape->d.embed > 0) {
            char *dz = take((size_t)mb * shape->d.embed * sizeof(bf16));
            if (m) m->dze = (bf16 *)dz;
        }
        if (shape->d.norm) {
            int cmax = 0;
            for (int l = 1; l <= shape->L; ++l) cmax = shape->Cs[l] > cmax ? shape->Cs[l] : cmax;
            const size_t lc = (size_t)4 * sms * 2 * cmax;
            char *lp2 = take(lc * sizeof(float));
            if (m) { m->ln_part = (float *)lp2; m->ln_cap = lc; }
        }
    }
    return off;
}

extern "C" size_t ppo_model_workspace_bytes(const ppo_model *m, int microbatch) {
    if (!m || microbatch <= 0) return 0;
    return carve(nullptr, m, microbatch, nullptr);
}

extern "C" int ppo_model_bind(ppo_model *m, float *master, void *shadow, float *grad, float *am, float *av, void *ws,
                              size_t ws_bytes, int microbatch) {
    if (!m || !master || !shadow || !grad || !am || !av || !ws || microbatch <= 0) return PPO_ERR_INVALID_ARG;
    if (!ppo_aligned(master, 16) || !ppo_aligned(shadow, 16) || !ppo_aligned(grad, 16) || !ppo_aligned(am, 16) ||
        !ppo_aligned(av, 16) || !ppo_aligned(ws, 256))
        return PPO_ERR_ALIGN;
    if (ws_bytes < ppo_model_workspace_bytes(m, microbatch)) return PPO_ERR_SHAPE;
    m->master = master;
    m->shadow = static_cast<bf16 *>(shadow);
    m->grad = grad;
    m->adam_m = am;
    m->adam_v = av;
    m->ws = static_cast<char *>(ws);
    m->ws_bytes = ws_bytes;
    m->mbmax = microbatch;
    carve(m, m, microbatch, m->ws);
    m->fwd_valid = false;
    m->wT_valid = false;
    return PPO_OK;
}

extern "C" int ppo_model_activation_ptr(const ppo_model *m, int kind, int index, void **ptr, size_t *elems) {
    if (!m || !ptr || !elems) return PPO_ERR_INVALID_ARG;
    if (!m->ws) return PPO_ERR_STATE;
    if (kind == 0 && index >= 1 && index <= m->L) {
        *ptr = m->act[index];
        *elems = (size_t)m->mbmax * m->Hs[index] * m->Ws[index] * m->Cs[index];
        return PPO_OK;
    }
    if (kind == 3 && index >= 1 && index <= m->L && m->xhat[index]) {
        *ptr = m->xhat[index];
        *elems = (size_t)m->mbmax * m->Hs[index] * m->Ws[index] * m->Cs[index];
        return PPO_OK;
    }
    if (kind == 4 && index >= 1 && index <= m->L && m->rstd[index]) {
        *ptr = m->rstd[index];
        *elems = (size_t)m->mbmax * m->Hs[index] * m->Ws[index];
        return PPO_OK;
    }
    if (kind >= 5 && kind <= 8 && index >= 0 && index < m->d.n_lstm) {
        const size_t H = (size_t)m->d.lstm_h, R = (size_t)m->mbmax;
        *ptr = kind == 5 ? (void *)m->lstm_hs[index] : kind == 6 ? (void *)m->lstm_c[index]
               : kind == 7 ? (void *)m->lstm_gates[index] : (void *)m->lstm_hprev[index];
        *elems = kind == 6 ? 2 * R * H : kind == 7 ? 4 * R * H : R * H;
        return PPO_OK;
    }
    if (kind == 2 && index >= 1 && index < m->L && m->abits[index]) {
        *ptr = m->abits[index];
        *elems = (size_t)m->mbmax * m->Hs[index] * m->Ws[index] * m->Cs[index] / 32;
        return PPO_OK;
    }
    if (kind == 1 && index >= 0 && index <= m->F) {
        *ptr = m->h[index];
        *elems = (size_t)m->mbmax * m->hw[index];
        return PPO_OK;
    }
    return PPO_ERR_INVALID_ARG;
}

extern "C" int ppo_model_set_sequence(ppo_model *m, int T, int Be, const uint8_t *done, const float *h_init,
                                      const float *c_init) {
    if (!m || !done || !h_init || !c_init) return PPO_ERR_INVALID_ARG;
    if (m->d.n_lstm == 0 || !m->ws) return PPO_ERR_STATE;
    if (T <= 0 || Be <= 0 || (long long)T * Be > m->mbmax) return PPO_ERR_SHAPE;
    m->seq_T = T;
    m->seq_Be = Be;
    m->seq_done = done;
    m->seq_h_init = h_init;
    m->seq_c_init = c_init;
    m->fwd_valid = false;
    return PPO_OK;
}

// h (bf16 -> fp32) and c of the last time step, zero where done: one thread per state element of a layer.
__global__ void __launch_bounds__(256) lstm_read_state_kernel(const bf16 *__restrict__ h, const float *__restrict__ c,
                                                              const uint8_t *__restrict__ done, float *__restrict__ h_out,
                                                              float *__restrict__ c_out, int Be, int H) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Be * H) return;
    const bool reset = done[i / H] != 0;
    h_out[i] = reset ? 0.f : __bfloat162float(h[i]);
    c_out[i] = reset ? 0.f : c[i];
}

extern "C" int ppo_model_read_state(const ppo_model *m, float *h_out, float *c_out, void *stream) {
    if (!m || !h_out || !c_out) return PPO_ERR_INVALID_ARG;
    if (m->d.n_lstm == 0 || !m->ws || m->seq_T <= 0 || !m->fwd_valid) return PPO_ERR_STATE;
    const int Be = m->seq_Be, H = m->d.lstm_h;
    const size_t last = (size_t)(m->seq_T - 1) * Be;
    for (int l = 0; l < m->d.n_lstm; ++l) {
        lstm_read_state_kernel<<<ppo_cdiv((long long)Be * H, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
            m->lstm_hs[l] + last * H, m->lstm_c[l] + last * H, m->seq_done + last, h_out + (size_t)l * Be * H,
            c_out + (size_t)l * Be * H, Be, H);
        PPO_LAUNCH_CHECK();
    }
    return PPO_OK;
}

extern "C" int ppo_model_sync_masks(ppo_model *m, int rows, void *stream) {
    if (!m || !m->ws) return PPO_ERR_STATE;
    if (rows <= 0 || rows > m->mbmax) return PPO_ERR_SHAPE;
    for (int l = 1; l < m->L; ++l)
        if (m->abits[l]) {
            const int s = relu_bits(m->act[l], m->abits[l], (long long)rows * m->Hs[l] * m->Ws[l], m->Cs[l],
                                    static_cast<cudaStream_t>(stream));
            if (s != PPO_OK) return s;
        }
    return PPO_OK;
}

// ------------------------------------------------------------ shadow / zero ----

__global__ void __launch_bounds__(256) shadow_kernel(const float4 *__restrict__ master, uint2 *__restrict__ shadow,
                                                     size_t n4) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    float4 x = master[i];
    __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y), hi = __floats2bfloat162_rn(x.z, x.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t *>(&lo);
    o.y = *reinterpret_cast<uint32_t *>(&hi);
    shadow[i] = o;
}

extern "C" int ppo_model_sync_shadow(ppo_model *m, void *stream) {
    if (!m || !m->master) return PPO_ERR_STATE;
    size_t n4 = m->arena / 4;
    shadow_kernel<<<ppo_cdiv(n4, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const float4 *>(m->master), reinterpret_cast<uint2 *>(m->shadow), n4);
    PPO_LAUNCH_CHECK();
    m->wT_valid = false;
    return PPO_OK;
}

extern "C" int ppo_model_zero_grad(ppo_model *m, void *stream) {
    if (!m || !m->grad) return PPO_ERR_STATE;
    PPO_CUDA_CHECK(cudaMemsetAsync(m->grad, 0, m->arena * sizeof(float), static_cast<cudaStream_t>(stream)));
    ppo_count_launches(1);
    return PPO_OK;
}

// -------------------------------------------------------------------- Adam ----

// One 128-bit lane per thread over the whole arena: reads theta, m, v, g (16 B/param),
// writes theta, m, v (12 B/param) and the bf16 shadow (2 B/param).
__global__ void __launch_bounds__(256) adam_kernel(float4 *__restrict__ theta, float4 *__restrict__ m,
                                                   float4 *__restrict__ v, const float4 *__restrict__ g,
                                                   uint2 *__restrict__ shadow, size_t n4, float lr, float b1,
                                                   float b2, float eps, float inv_c1, float inv_c2) {
    const size_t nth = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += nth) {
        float4 th = theta[i], mm = m[i], vv = v[i];
        const float4 gg = g[i];
        float *pt = &th.x, *pm = &mm.x, *pv = &vv.x;
        const float *pg = &gg.x;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            pm[j] = b1 * pm[j] + (1.f - b1) * pg[j];
            pv[j] = b2 * pv[j] + (1.f - b2) * pg[j] * pg[j];
            const float mhat = pm[j] * inv_c1, vhat = pv[j] * inv_c2;
            pt[j] = pt[j] - lr * mhat / (sqrtf(vhat) + eps);
        }
        theta[i] = th;
        m[i] = mm;
        v[i] = vv;
        __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y), hi = __floats2bfloat162_rn(th.z, th.w);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t *>(&lo);
        o.y = *reinterpret_cast<uint32_t *>(&hi);
        shadow[i] = o;
    }
}

extern "C" int ppo_adam_step(ppo_model *m, float lr, float beta1, float beta2, float eps, int64_t step,
                             void *stream) {
    if (!m || !m->master) return PPO_ERR_STATE;
    if (step < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps > 0.f))
        return PPO_ERR_INVALID_ARG;
    const double c1 = 1.0 - pow((double)beta1, (double)step), c2 = 1.0 - pow((double)beta2, (double)step);
    const size_t n4 = m->arena / 4;
    int blocks = ppo_cdiv(n4, 256);
    const int cap = ppo_num_sms() * 8;
    if (blocks > cap) blocks = cap;
    adam_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<float4 *>(m->master), reinterpret_cast<float4 *>(m->adam_m),
        reinterpret_cast<float4 *>(m->adam_v), reinterpret_cast<const float4 *>(m->grad),
        reinterpret_cast<uint2 *>(m->shadow), n4, lr, beta1, beta2, eps, (float)(1.0 / c1), (float)(1.0 / c2));
    PPO_LAUNCH_CHECK();
    m->wT_valid = false;
    m->fwd_valid = false;
    return PPO_OK;
}

// -------------------------------------------------------------------- loss ----

#define PPO_MAX_A 16
#define PPO_HALF_LOG_2PI 0.91893853320467274178f

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// One thread per row: log-prob, ratio, clipped surrogate, value error and their gradients.
// Block sums of {L_pi, L_V, kl, clipfrac, dlogsigma[A]} go to partials[blockIdx.x][32].
__global__ void __launch_bounds__(kLossThreads) loss_kernel(
    int rows, int A, float inv_Bt, const float *__restrict__ mean, const float *__restrict__ value,
    const float *__restrict__ logsigma, const float *__restrict__ action, const float *__restrict__ logp_old,
    const float *__restrict__ adv, const float *__restrict__ ret, float clip, float vf_coef,
    float *__restrict__ dmean, float *__restrict__ dvalue, float *__restrict__ partials) {
    __shared__ float sh[kLossThreads / 32][4 + PPO_MAX_A];
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    float acc[4 + PPO_MAX_A];
#pragma unroll
    for (int j = 0; j < 4 + PPO_MAX_A; ++j) acc[j] = 0.f;
    if (i < rows) {
        float z[PPO_MAX_A], inv_sg[PPO_MAX_A];
        float logp = 0.f;
#pragma unroll
        for (int j = 0; j < PPO_MAX_A; ++j) {
            if (j < A) {
                const float ls = logsigma[j];
                inv_sg[j] = expf(-ls);
                z[j] = (action[(size_t)i * A + j] - mean[(size_t)i * A + j]) * inv_sg[j];
                logp += -0.5f * z[j] * z[j] - ls - PPO_HALF_LOG_2PI;
            }
        }
        const float lpo = logp_old[i];
        const float r = expf(logp - lpo);
        const float rc = fminf(fmaxf(r, 1.f - clip), 1.f + clip);
        const float a = adv[i];
        const float s_un = r * a, s_cl = rc * a;
        const bool unclipped = s_un <= s_cl;
        const float s = unclipped ? s_un : s_cl;
        const float gs = unclipped ? a : 0.f;
        const float verr = value[i] - ret[i];
        acc[0] = -s * inv_Bt;
        acc[1] = verr * verr * inv_Bt;
        acc[2] = (lpo - logp) * inv_Bt;
        acc[3] = (fabsf(r - 1.f) > clip ? 1.f : 0.f) * inv_Bt;
        const float dlogp = -gs * r * inv_Bt;
#pragma unroll
        for (int j = 0; j < PPO_MAX_A; ++j) {
            if (j < A) {
                dmean[(size_t)i * A + j] = dlogp * z[j] * inv_sg[j];
                acc[4 + j] = dlogp * (z[j] * z[j] - 1.f);
            }
        }
        dvalue[i] = 2.f * vf_coef * verr * inv_Bt;
    }
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < 4 + PPO_MAX_A; ++j) {
        float v = warp_sum_f(acc[j]);
        if (lane == 0) sh[wid][j] = v;
    }
    __syncthreads();
    if (threadIdx.x < 4 + PPO_MAX_A) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < kLossThreads / 32; ++w) v += sh[w][threadIdx.x];
        partials[(size_t)blockIdx.x * 32 + threadIdx.x] = v;
    }
}

// Single block: fixed-order sum of the per-block partials (fp64), added into the loss
// scalars and the log-sigma gradient.
__global__ void __launch_bounds__(32) loss_finalize_kernel(const float *__restrict__ partials, int nblocks, int A,
                                                           const float *__restrict__ logsigma, float share,
                                                           float ent_coef, float *__restrict__ loss_out,
                                                           float *__restrict__ grad_logsigma) {
    const int j = threadIdx.x;
    if (j >= 4 + A) return;
    double s = 0.0;
    for (int b = 0; b < nblocks; ++b) s += (double)partials[(size_t)b * 32 + j];
    if (j == 0) loss_out[0] += (float)s;
    if (j == 1) loss_out[1] += (float)s;
    if (j == 2) loss_out[3] += (float)s;
    if (j == 3) loss_out[4] += (float)s;
    if (j >= 4) grad_logsigma[j - 4] += (float)s - ent_coef * share;
    if (j == 0) {
        float H = 0.5f * A * (1.f + 2.f * PPO_HALF_LOG_2PI);
        for (int k = 0; k < A; ++k) H += logsigma[k];
        loss_out[2] += H * share;
    }
}

extern "C" int ppo_loss_fwd_bwd(ppo_model *m, const ppo_minibatch *mb, int row0, int rows, int B_total,
                                const float *mean, const float *value, float clip, float vf_coef, float ent_coef,
                                float *loss_out, float *dmean, float *dvalue, void *stream) {
    if (!m || !mb || !mean || !value || !loss_out || !dmean || !dvalue) return PPO_ERR_INVALID_ARG;
    if (!m->master) return PPO_ERR_STATE;
    if (row0 < 0 || rows <= 0 || row0 + rows > mb->B || B_total < rows || rows > m->mbmax) return PPO_ERR_SHAPE;
    if (!(clip > 0.f)) return PPO_ERR_INVALID_ARG;
    const int A = m->d.A;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float *logsigma = m->master + m->tensors.back().off;
    const int blocks = ppo_cdiv(rows, kLossThreads);
    loss_kernel<<<blocks, kLossThreads, 0, st>>>(rows, A, 1.f / (float)B_total, mean, value, logsigma,
                                                 mb->action + (size_t)row0 * A, mb->logp_old + row0, mb->adv + row0,
                                                 mb->ret + row0, clip, vf_coef, dmean, dvalue, m->loss_partials);
    PPO_LAUNCH_CHECK();
    loss_finalize_kernel<<<1, 32, 0, st>>>(m->loss_partials, blocks, A, logsigma, (float)rows / (float)B_total,
                                           ent_coef, loss_out, m->grad + m->tensors.back().off);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

// ------------------------------------------------------------------ sample ----

__global__ void __launch_bounds__(128) sample_kernel(int rows, int A, const float *__restrict__ mean,
                                                     const float *__restrict__ logsigma,
                                                     const float *__restrict__ eps, float *__restrict__ action,
                                                     float *__restrict__ logp) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    float lp = 0.f;
    for (int j = 0; j < A; ++j) {
        const float ls = logsigma[j], e = eps[(size_t)i * A + j];
        action[(size_t)i * A + j] = mean[(size_t)i * A + j] + expf(ls) * e;
        lp += -0.5f * e * e - ls - PPO_HALF_LOG_2PI;
    }
    logp[i] = lp;
}

extern "C" int ppo_policy_sample(const ppo_model *m, int rows, const float *mean, const float *eps, float *action,
                                 float *logp, void *stream) {
    if (!m || !mean || !eps || !action || !logp || rows <= 0) return PPO_ERR_INVALID_ARG;
    if (!m->master) return PPO_ERR_STATE;
    sample_kernel<<<ppo_cdiv(rows, 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        rows, m->d.A, mean, m->master + m->tensors.back().off, eps, action, logp);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

// actions <- pi(obs) for time step t of the buffer, in place: the observation is read from slab row t and the
// action, its log-density and the value estimate are written into slab row t.
extern "C" int ppo_policy_act(ppo_model *m, ppo_buffer *b, int t, const float *eps, void *stream) {
    if (!m || !b || !eps) return PPO_ERR_INVALID_ARG;
    if (!m->master) return PPO_ERR_STATE;
    const ppo_buffer_desc &d = b->d;
    if (t < 0 || t >= d.T) return PPO_ERR_INVALID_ARG;
    if (d.H != m->d.H || d.W != m->d.W || d.P != m->d.P || d.A != m->d.A) return PPO_ERR_SHAPE;
    if (m->d.n_lstm > 0) return PPO_ERR_UNSUPPORTED;  // a recurrent policy acts through ppo_model_set_sequence + ppo_encoder_fwd
    const size_t N = (size_t)d.N;
    char *depth = b->base + b->field_off[PPO_FIELD_DEPTH] + (size_t)t * N * d.H * d.W * 2;
    float *proprio = reinterpret_cast<float *>(b->base + b->field_off[PPO_FIELD_PROPRIO]) + (size_t)t * N * d.P;
    float *action = reinterpret_cast<float *>(b->base + b->field_off[PPO_FIELD_ACTION]) + (size_t)t * N * d.A;
    float *logp = reinterpret_cast<float *>(b->base + b->field_off[PPO_FIELD_LOGP]) + (size_t)t * N;
    float *value = reinterpret_cast<float *>(b->base + b->field_off[PPO_FIELD_VALUE]) + (size_t)t * N;
    ppo_minibatch obs = {};
    obs.depth_f16 = depth;
    obs.proprio = proprio;
    obs.B = d.N;
    b->gae_valid = false;
    for (int r0 = 0; r0 < d.N; r0 += m->mbmax) {
        const int rows = d.N - r0 < m->mbmax ? d.N - r0 : m->mbmax;
        int s = ppo_encoder_fwd(m, &obs, r0, rows, m->act_mean, value + r0, stream);
        if (s != PPO_OK) return s;
        s = ppo_policy_sample(m, rows, m->act_mean, eps + (size_t)r0 * d.A, action + (size_t)r0 * d.A, logp + r0, stream);
        if (s != PPO_OK) return s;
    }
    m->fwd_valid = false;  // these activations belong to no minibatch a backward pass could name
    return PPO_OK;
}
