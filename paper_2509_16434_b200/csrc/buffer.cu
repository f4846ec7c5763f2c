// Rollout buffer D on the learner GPU (Algorithm 2): slab carving, write_step, GAE with
// advantage normalisation, and the seeded permutation gather.
#include <atomic>
#include <new>

#include "common.cuh"

// ------------------------------------------------------------------ status ----

static __device__ int32_t g_ppo_status;

int32_t *ppo_device_status_ptr() {
    static int32_t *ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!ptrs[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_ppo_status) != cudaSuccess) return nullptr;
        ptrs[dev] = static_cast<int32_t *>(p);
    }
    return ptrs[dev];
}

static std::atomic<unsigned long long> g_launches{0};

void ppo_count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

extern "C" uint64_t ppo_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int ppo_num_sms() {
    static int sms[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!sms[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        sms[dev] = n;
    }
    return sms[dev];
}

extern "C" const char *ppo_status_string(int s) {
    switch (s) {
        case PPO_OK: return "ok";
        case PPO_ERR_INVALID_ARG: return "invalid argument";
        case PPO_ERR_SHAPE: return "shape mismatch";
        case PPO_ERR_ALIGN: return "misaligned pointer";
        case PPO_ERR_STATE: return "call out of order";
        case PPO_ERR_CUDA: return "CUDA error";
        case PPO_ERR_TIMEOUT: return "device-side wait timed out";
        case PPO_ERR_UNSUPPORTED: return "unsupported shape";
        default: return "unknown status";
    }
}

extern "C" int ppo_poll_status(void *stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *p = ppo_device_status_ptr();
    if (!p) return PPO_ERR_CUDA;
    int32_t host = 0;
    if (cudaMemcpyAsync(&host, p, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess) return PPO_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PPO_ERR_CUDA;
    if (host != 0) {
        if (cudaMemsetAsync(p, 0, sizeof(host), st) != cudaSuccess) return PPO_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return PPO_ERR_CUDA;
    }
    return host;
}

// ------------------------------------------------------------------ layout ----

static const int kMaxGaeBlocks = 4096;

static bool desc_ok(const ppo_buffer_desc *d) {
    return d && d->N > 0 && d->T > 0 && d->H > 0 && d->W > 0 && d->P > 0 && d->A > 0 &&
           (long long)d->N * d->T < (1ll << 31);
}

static size_t field_bytes(const ppo_buffer_desc *d, int field, int depth_elem) {
    size_t M = (size_t)d->N * d->T;
    switch (field) {
        case PPO_FIELD_DEPTH: return M * d->H * d->W * (size_t)depth_elem;
        case PPO_FIELD_PROPRIO: return M * d->P * 4;
        case PPO_FIELD_ACTION: return M * d->A * 4;
        case PPO_FIELD_LOGP:
        case PPO_FIELD_VALUE:
        case PPO_FIELD_REWARD:
        case PPO_FIELD_ADV:
        case PPO_FIELD_RET: return M * 4;
        case PPO_FIELD_DONE: return M;
        case PPO_FIELD_SCRATCH: return (size_t)kMaxGaeBlocks * 2 * sizeof(double);
        default: return 0;
    }
}

extern "C" size_t ppo_buffer_field_bytes(const ppo_buffer_desc *d, int field, int depth_elem_bytes) {
    if (!desc_ok(d) || field < 0 || field >= PPO_NUM_FIELDS) return 0;
    if (depth_elem_bytes != 2 && depth_elem_bytes != 4) return 0;
    return field_bytes(d, field, depth_elem_bytes);
}

extern "C" size_t ppo_buffer_bytes(const ppo_buffer_desc *d) {
    if (!desc_ok(d)) return 0;
    size_t total = 0;
    for (int f = 0; f < PPO_NUM_FIELDS; ++f) total += ppo_align_up(field_bytes(d, f, 2), 256);
    return total;
}

extern "C" int ppo_buffer_alloc(const ppo_buffer_desc *d, void *dev_storage, size_t bytes, ppo_buffer **out) {
    if (!out) return PPO_ERR_INVALID_ARG;
    *out = nullptr;
    if (!desc_ok(d) || !dev_storage) return PPO_ERR_INVALID_ARG;
    if (!ppo_aligned(dev_storage, 256)) return PPO_ERR_ALIGN;
    if (bytes < ppo_buffer_bytes(d)) return PPO_ERR_SHAPE;
    ppo_buffer *b = new (std::nothrow) ppo_buffer();
    if (!b) return PPO_ERR_INVALID_ARG;
    b->d = *d;
    b->base = static_cast<char *>(dev_storage);
    b->bytes = bytes;
    size_t off = 0;
    for (int f = 0; f < PPO_NUM_FIELDS; ++f) {
        b->field_off[f] = off;
        off += ppo_align_up(field_bytes(d, f, 2), 256);
    }
    b->gae_valid = false;
    b->gae_blocks = 0;
    b->barrier_zeroed = false;
    *out = b;
    return PPO_OK;
}

extern "C" int ppo_buffer_free(ppo_buffer *b) {
    if (!b) return PPO_ERR_INVALID_ARG;
    delete b;
    return PPO_OK;
}

extern "C" void *ppo_buffer_field_ptr(const ppo_buffer *b, int field) {
    if (!b || field < 0 || field >= PPO_NUM_FIELDS) return nullptr;
    return b->base + b->field_off[field];
}

template <typename T>
static T *slab(const ppo_buffer *b, int field) {
    return reinterpret_cast<T *>(b->base + b->field_off[field]);
}

// -------------------------------------------------------------- write_step ----

struct CopySeg {
    const char *src;
    char *dst;
    unsigned long long bytes;
    int vec;  // 16 when both ends and the size allow 128-bit accesses, else 1
};
struct CopySegs {
    CopySeg s[7];
};

// blockIdx.y selects the segment; blocks stride over it with 128-bit (or byte) accesses.
__global__ void __launch_bounds__(256) write_step_kernel(CopySegs segs) {
    const CopySeg sg = segs.s[blockIdx.y];
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nth = (unsigned long long)gridDim.x * blockDim.x;
    if (sg.vec == 16) {
        const uint4 *s = reinterpret_cast<const uint4 *>(sg.src);
        uint4 *d = reinterpret_cast<uint4 *>(sg.dst);
        const unsigned long long n = sg.bytes >> 4;
        unsigned long long i = tid;
        for (; i + 3 * nth < n; i += 4 * nth) {
            uint4 a = __ldcs(s + i), b = __ldcs(s + i + nth), c = __ldcs(s + i + 2 * nth), e = __ldcs(s + i + 3 * nth);
            d[i] = a;
            d[i + nth] = b;
            d[i + 2 * nth] = c;
            d[i + 3 * nth] = e;
        }
        for (; i < n; i += nth) d[i] = __ldcs(s + i);
    } else {
        for (unsigned long long i = tid; i < sg.bytes; i += nth) sg.dst[i] = sg.src[i];
    }
}

// Copies up to 7 per-env arrays of one step into slab row t (null sources are skipped).
static int write_fields(ppo_buffer *b, int t, const void *const srcs[7], void *stream) {
    const ppo_buffer_desc &d = b->d;
    const size_t N = d.N;
    const int fields[7] = {PPO_FIELD_DEPTH, PPO_FIELD_PROPRIO, PPO_FIELD_ACTION, PPO_FIELD_LOGP,
                           PPO_FIELD_VALUE, PPO_FIELD_REWARD, PPO_FIELD_DONE};
    const size_t per_env[7] = {(size_t)d.H * d.W * 2, (size_t)d.P * 4, (size_t)d.A * 4, 4, 4, 4, 1};
    CopySegs segs;
    int n = 0;
    size_t largest = 0;
    for (int i = 0; i < 7; ++i) {
        if (!srcs[i]) continue;
        size_t bytes = N * per_env[i];
        char *dst = b->base + b->field_off[fields[i]] + (size_t)t * bytes;
        segs.s[n].src = static_cast<const char *>(srcs[i]);
        segs.s[n].dst = dst;
        segs.s[n].bytes = bytes;
        segs.s[n].vec = (ppo_aligned(srcs[i], 16) && ppo_aligned(dst, 16) && bytes % 16 == 0) ? 16 : 1;
        largest = bytes > largest ? bytes : largest;
        ++n;
    }
    b->gae_valid = false;
    if (n == 0) return PPO_OK;
    // enough blocks to cover the largest segment with ~4 x 16 B per thread, capped at a few waves
    long long units = (long long)(largest / 16 / 4 / 256) + 1;
    int gx = (int)(units < (long long)ppo_num_sms() * 16 ? units : (long long)ppo_num_sms() * 16);
    dim3 grid(gx, n);
    write_step_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(segs);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

extern "C" int ppo_buffer_write_step(ppo_buffer *b, int t, const void *depth, const float *proprio,
                                     const float *action, const float *logp, const float *value, const float *reward,
                                     const uint8_t *done, void *stream) {
    if (!b || !depth || !proprio || !action || !logp || !value || !reward || !done) return PPO_ERR_INVALID_ARG;
    if (t < 0 || t >= b->d.T) return PPO_ERR_INVALID_ARG;
    const void *srcs[7] = {depth, proprio, action, logp, value, reward, done};
    return write_fields(b, t, srcs, stream);
}

extern "C" int ppo_buffer_write_obs(ppo_buffer *b, int t, const void *depth, const float *proprio, void *stream) {
    if (!b || !depth || !proprio) return PPO_ERR_INVALID_ARG;
    if (t < 0 || t >= b->d.T) return PPO_ERR_INVALID_ARG;
    const void *srcs[7] = {depth, proprio, nullptr, nullptr, nullptr, nullptr, nullptr};
    return write_fields(b, t, srcs, stream);
}

extern "C" int ppo_buffer_write_outcome(ppo_buffer *b, int t, const float *reward, const uint8_t *done, void *stream) {
    if (!b || !reward || !done) return PPO_ERR_INVALID_ARG;
    if (t < 0 || t >= b->d.T) return PPO_ERR_INVALID_ARG;
    const void *srcs[7] = {nullptr, nullptr, nullptr, nullptr, nullptr, reward, done};
    return write_fields(b, t, srcs, stream);
}

// --------------------------------------------------------------------- GAE ----

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block; the result is valid in thread 0.  Fixed reduction order.
__device__ __forceinline__ double block_sum(double v, double *sh /*[32]*/) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    if (wid == 0) {
        v = (lane < (int)((blockDim.x + 31) >> 5)) ? sh[lane] : 0.0;
        v = warp_sum(v);
    }
    return v;
}

// One thread per env: reverse scan over t with the loads of UNR steps issued together.
// Reads r, V (fp32) and d (u8), writes A and R: 17 B per env-step.  Each block leaves the
// fp64 sums of A and A^2 of its envs in partials[2*blockIdx.x .. +1].
template <int UNR>
__global__ void __launch_bounds__(128) gae_scan_kernel(const float *__restrict__ reward,
                                                       const float *__restrict__ value,
                                                       const uint8_t *__restrict__ done,
                                                       const float *__restrict__ last_value, float gamma,
                                                       float gamma_lambda, float *__restrict__ adv,
                                                       float *__restrict__ ret, int T, int N,
                                                       double *__restrict__ partials) {
    __shared__ double sh[32];
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    double s1 = 0.0, s2 = 0.0;
    if (n < N) {
        float v_next = last_value[n];
        float a_next = 0.f;
        int t = T - 1;
        for (; t >= UNR - 1; t -= UNR) {
            float r[UNR], v[UNR];
            uint8_t d[UNR];
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                size_t i = (size_t)(t - u) * N + n;
                r[u] = __ldcs(reward + i);
                v[u] = __ldcs(value + i);
                d[u] = __ldcs(done + i);
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                size_t i = (size_t)(t - u) * N + n;
                float nd = d[u] ? 0.f : 1.f;
                float delta = r[u] + gamma * v_next * nd - v[u];
                float a = delta + gamma_lambda * nd * a_next;
                __stcs(adv + i, a);
                __stcs(ret + i, a + v[u]);
                s1 += (double)a;
                s2 += (double)a * (double)a;
                v_next = v[u];
                a_next = a;
            }
        }
        for (; t >= 0; --t) {
            size_t i = (size_t)t * N + n;
            float r = reward[i], v = value[i];
            float nd = done[i] ? 0.f : 1.f;
            float delta = r + gamma * v_next * nd - v;
            float a = delta + gamma_lambda * nd * a_next;
            adv[i] = a;
            ret[i] = a + v;
            s1 += (double)a;
            s2 += (double)a * (double)a;
            v_next = v;
            a_next = a;
        }
    }
    s1 = block_sum(s1, sh);
    s2 = block_sum(s2, sh);
    if (threadIdx.x == 0) {
        partials[2 * blockIdx.x] = s1;
        partials[2 * blockIdx.x + 1] = s2;
    }
}

// Every block reduces the per-block partial sums in the same fixed order (deterministic),
// then normalises its share of the advantages in place with 128-bit accesses.
__global__ void __launch_bounds__(256) adv_normalize_kernel(float *__restrict__ adv, long long M,
                                                            const double *__restrict__ partials, int nparts,
                                                            float *__restrict__ stats_out) {
    __shared__ double sh[32];
    __shared__ float s_mean, s_inv;
    double s1 = 0.0, s2 = 0.0;
    for (int i = threadIdx.x; i < nparts; i += blockDim.x) {
        s1 += partials[2 * i];
        s2 += partials[2 * i + 1];
    }
    s1 = block_sum(s1, sh);
    s2 = block_sum(s2, sh);
    if (threadIdx.x == 0) {
        double mean = s1 / (double)M;
        double var = (M > 1) ? (s2 - s1 * mean) / (double)(M - 1) : 0.0;
        double sd = sqrt(var > 0.0 ? var : 0.0);
        s_mean = (float)mean;
        s_inv = (float)(1.0 / (sd + 1e-8));
        if (blockIdx.x == 0 && stats_out) {
            stats_out[0] = (float)mean;
            stats_out[1] = (float)sd;
        }
    }
    __syncthreads();
    const float mean = s_mean, inv = s_inv;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nth = (long long)gridDim.x * blockDim.x;
    const long long n4 = M >> 2;
    float4 *a4 = reinterpret_cast<float4 *>(adv);
    for (long long i = tid; i < n4; i += nth) {
        float4 x = a4[i];
        x.x = (x.x - mean) * inv;
        x.y = (x.y - mean) * inv;
        x.z = (x.z - mean) * inv;
        x.w = (x.w - mean) * inv;
        a4[i] = x;
    }
    for (long long i = (n4 << 2) + tid; i < M; i += nth) adv[i] = (adv[i] - mean) * inv;
}

// GAE, the moments of the advantages and their normalisation in ONE launch, for buffers whose scan blocks are all
// resident at once (cooperative launch): scan as gae_scan_kernel does, a grid barrier, then every block reduces the
// per-block partial sums in the same fixed order and normalises the advantages of its own envs (which it wrote
// itself).  The barrier is a counter that wraps to zero on the last arrival (so it needs no reset) and a generation
// word the last arriver bumps; its wait is bounded: on a time-out the block records PPO_ERR_TIMEOUT and returns
// without normalising.
__global__ void __launch_bounds__(128) gae_fused_kernel(const float *__restrict__ reward, const float *__restrict__ value,
                                                        const uint8_t *__restrict__ done,
                                                        const float *__restrict__ last_value, float gamma,
                                                        float gamma_lambda, float *__restrict__ adv,
                                                        float *__restrict__ ret, int T, int N, double *partials,
                                                        unsigned int *barrier /*[2]: counter, generation*/,
                                                        float *__restrict__ stats_out, int32_t *status) {
    __shared__ double sh[32];
    __shared__ float s_mean, s_inv;
    __shared__ int s_ok;
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    double s1 = 0.0, s2 = 0.0;
    if (n < N) {
        float v_next = last_value[n], a_next = 0.f;
        for (int t = T - 1; t >= 0; --t) {
            const size_t i = (size_t)t * N + n;
            const float r = __ldcs(reward + i), v = __ldcs(value + i);
            const float nd = __ldcs(done + i) ? 0.f : 1.f;
            const float delta = r + gamma * v_next * nd - v;
            const float a = delta + gamma_lambda * nd * a_next;
            adv[i] = a;
            ret[i] = a + v;
            s1 += (double)a;
            s2 += (double)a * (double)a;
            v_next = v;
            a_next = a;
        }
    }
    s1 = block_sum(s1, sh);
    s2 = block_sum(s2, sh);
    if (threadIdx.x == 0) {
        partials[2 * blockIdx.x] = s1;
        partials[2 * blockIdx.x + 1] = s2;
        __threadfence();
        volatile unsigned int *gen = barrier + 1;
        const unsigned int my_gen = *gen;
        int ok = 1;
        if (atomicInc(barrier, gridDim.x - 1) == gridDim.x - 1) {
            __threadfence();
            atomicAdd(barrier + 1, 1u);
        } else {
            const long long t0 = clock64();
            while (*gen == my_gen) {
                if (clock64() - t0 > 2000000000ll) {  // ~1 s
                    ppo_report(status, PPO_ERR_TIMEOUT);
                    ok = 0;
                    break;
                }
            }
        }
        __threadfence();
        s_ok = ok;
    }
    __syncthreads();
    if (!s_ok) return;
    const long long M = (long long)N * T;
    double t1 = 0.0, t2 = 0.0;
    for (int i = threadIdx.x; i < (int)gridDim.x; i += blockDim.x) {
        t1 += __ldcg(partials + 2 * i);
        t2 += __ldcg(partials + 2 * i + 1);
    }
    t1 = block_sum(t1, sh);
    t2 = block_sum(t2, sh);
    if (threadIdx.x == 0) {
        const double mean = t1 / (double)M;
        const double var = (M > 1) ? (t2 - t1 * mean) / (double)(M - 1) : 0.0;
        const double sd = sqrt(var > 0.0 ? var : 0.0);
        s_mean = (float)mean;
        s_inv = (float)(1.0 / (sd + 1e-8));
        if (blockIdx.x == 0 && stats_out) {
            stats_out[0] = (float)mean;
            stats_out[1] = (float)sd;
        }
    }
    __syncthreads();
    if (n < N) {
        const float mean = s_mean, inv = s_inv;
        for (int t = 0; t < T; ++t) {
            const size_t i = (size_t)t * N + n;
            adv[i] = (adv[i] - mean) * inv;
        }
    }
}

// Blocks of gae_fused_kernel that can be resident at once on the current device (0: cooperative launch unavailable).
static int gae_fused_capacity() {
    static int cap[64] = {0};
    static bool known[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!known[dev]) {
        int coop = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && coop &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, gae_fused_kernel, 128, 0) == cudaSuccess)
            cap[dev] = per_sm * ppo_num_sms();
        known[dev] = true;
    }
    return cap[dev];
}

extern "C" int ppo_compute_gae(ppo_buffer *b, const float *last_value, float gamma, float lambda, int normalize,
                               float *stats_out, void *stream) {
    if (!b || !last_value) return PPO_ERR_INVALID_ARG;
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f)) return PPO_ERR_INVALID_ARG;
    const int N = b->d.N, T = b->d.T;
    const int threads = 128;
    const int blocks = ppo_cdiv(N, threads);
    if (blocks > kMaxGaeBlocks) return PPO_ERR_UNSUPPORTED;  // N <= 524288 envs
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double *partials = slab<double>(b, PPO_FIELD_SCRATCH);
    // normalize == 2: one cooperative launch, possible when the whole scan is resident at once (every configuration
    // of the workloads).  Measured, it is no faster than the two plain launches (24 against 18 microseconds at 1024
    // envs x 16 steps: a cooperative launch and its grid barrier cost more than the second launch they save), so it
    // is an option, not the default.  The last 8 bytes of the scratch slab hold the grid barrier; they are free
    // while blocks < kMaxGaeBlocks.
    if (normalize == 2 && (blocks >= kMaxGaeBlocks || blocks > gae_fused_capacity())) return PPO_ERR_UNSUPPORTED;
    if (normalize == 2) {
        unsigned int *barrier = reinterpret_cast<unsigned int *>(partials + 2 * kMaxGaeBlocks) - 2;
        if (!b->barrier_zeroed) {
            PPO_CUDA_CHECK(cudaMemsetAsync(barrier, 0, 8, st));
            ppo_count_launches(1);
            b->barrier_zeroed = true;
        }
        const float *reward = slab<float>(b, PPO_FIELD_REWARD), *value = slab<float>(b, PPO_FIELD_VALUE);
        const uint8_t *done = slab<uint8_t>(b, PPO_FIELD_DONE);
        float *adv = slab<float>(b, PPO_FIELD_ADV), *ret = slab<float>(b, PPO_FIELD_RET);
        float gl = gamma * lambda;
        int32_t *status = ppo_device_status_ptr();
        int Ti = T, Ni = N;
        void *args[] = {&reward, &value, &done, &last_value, &gamma, &gl, &adv, &ret, &Ti, &Ni, &partials, &barrier,
                        &stats_out, &status};
        PPO_CUDA_CHECK(cudaLaunchCooperativeKernel((const void *)gae_fused_kernel, dim3(blocks), dim3(threads), args, 0, st));
        PPO_LAUNCH_CHECK();
        b->gae_valid = true;
        b->gae_blocks = blocks;
        return PPO_OK;
    }
    gae_scan_kernel<8><<<blocks, threads, 0, st>>>(slab<float>(b, PPO_FIELD_REWARD), slab<float>(b, PPO_FIELD_VALUE),
                                                   slab<uint8_t>(b, PPO_FIELD_DONE), last_value, gamma,
                                                   gamma * lambda, slab<float>(b, PPO_FIELD_ADV),
                                                   slab<float>(b, PPO_FIELD_RET), T, N, partials);
    PPO_LAUNCH_CHECK();
    if (normalize) {
        const long long M = (long long)N * T;
        int nb = ppo_cdiv(M, 256 * 4 * 4);
        int cap = ppo_num_sms() * 8;
        if (nb > cap) nb = cap;
        if (nb < 1) nb = 1;
        adv_normalize_kernel<<<nb, 256, 0, st>>>(slab<float>(b, PPO_FIELD_ADV), M, partials, blocks, stats_out);
        PPO_LAUNCH_CHECK();
    }
    b->gae_valid = true;
    b->gae_blocks = blocks;
    return PPO_OK;
}

// ------------------------------------------------------------ GAE, no allocation ----

// Scratch of ppo_gae_static: the per-block partial sums the scan leaves for the normalisation pass.
// Lives in the library image, so every device that loads the library holds these 64 KB until exit.
static __device__ __align__(256) double g_gae_static_scratch[2 * kMaxGaeBlocks];

// Device address of the scratch array on the current device (nullptr on error).  The array's name is
// only a host-side handle; kernels must be given the address cudaGetSymbolAddress returns.
static double *gae_static_scratch_ptr() {
    static double *ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!ptrs[dev]) {
        double *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_gae_static_scratch) != cudaSuccess) return nullptr;
        ptrs[dev] = p;
    }
    return ptrs[dev];
}

extern "C" int ppo_gae_static(const float *reward, const float *value, const uint8_t *done, const float *last_value,
                              int T, int N, float gamma, float lambda, int normalize, float *adv, float *ret,
                              float *stats_out, void *stream) {
    if (!reward || !value || !done || !last_value || !adv || !ret) return PPO_ERR_INVALID_ARG;
    if (T <= 0 || N <= 0 || (long long)T * N >= (1ll << 31)) return PPO_ERR_INVALID_ARG;
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f)) return PPO_ERR_INVALID_ARG;
    if (N > PPO_GAE_STATIC_MAX_ENVS) return PPO_ERR_UNSUPPORTED;  // more envs than the fixed scratch covers
    if (!ppo_aligned(adv, 16)) return PPO_ERR_ALIGN;
    const int threads = 128;
    const int blocks = ppo_cdiv(N, threads);
    double *partials = gae_static_scratch_ptr();
    if (!partials) return PPO_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // every partial a later pass reads is written by this launch first: nothing has to start at zero
    gae_scan_kernel<8><<<blocks, threads, 0, st>>>(reward, value, done, last_value, gamma, gamma * lambda, adv, ret, T, N,
                                                   partials);
    PPO_LAUNCH_CHECK();
    if (normalize) {
        const long long M = (long long)N * T;
        int nb = ppo_cdiv(M, 256 * 4 * 4);
        const int cap = ppo_num_sms() * 8;
        nb = nb > cap ? cap : (nb < 1 ? 1 : nb);
        adv_normalize_kernel<<<nb, 256, 0, st>>>(adv, M, partials, blocks, stats_out);
        PPO_LAUNCH_CHECK();
    }
    return PPO_OK;
}

// ------------------------------------------------------------------ gather ----

struct PermParams {
    uint32_t key[6];
    uint32_t M;
    int h;
    uint32_t mask;
};

__host__ __device__ __forceinline__ uint32_t perm_mix(uint32_t x) {
    x ^= x >> 16;
    x *= 0x9E3779B9u;
    x ^= x >> 15;
    x *= 0x6A09E667u;
    x ^= x >> 16;
    return x;
}

static PermParams make_perm(uint64_t seed, uint32_t epoch, uint32_t M) {
    PermParams p;
    const uint32_t lo = (uint32_t)seed, hi = (uint32_t)(seed >> 32);
    for (uint32_t j = 0; j < 6; ++j)
        p.key[j] = perm_mix(lo ^ perm_mix(hi + 0x9E3779B9u * (j + 1)) ^ perm_mix(epoch + 0xBB67AE85u * (j + 1)));
    int bits = 0;
    while ((1ull << bits) < (unsigned long long)M) ++bits;
    p.h = (bits + 1) / 2 < 1 ? 1 : (bits + 1) / 2;
    p.mask = (1u << p.h) - 1u;
    p.M = M;
    return p;
}

__device__ __forceinline__ uint32_t perm_apply(const PermParams &p, uint32_t i) {
    uint32_t x = i;
    do {
        uint32_t L = x >> p.h, R = x & p.mask;
#pragma unroll
        for (int j = 0; j < 6; ++j) {
            uint32_t nr = L ^ (perm_mix(R ^ p.key[j]) & p.mask);
            L = R;
            R = nr;
        }
        x = (L << p.h) | R;
    } while (x >= p.M);
    return x;
}

struct GatherArgs {
    const char *depth;
    const float *proprio, *action, *logp, *value, *adv, *ret;
    char *o_depth;
    float *o_proprio, *o_action, *o_logp, *o_value, *o_adv, *o_ret;
    uint32_t *o_index;
    uint32_t start;      // first position of this minibatch in the permuted order
    uint32_t rows;       // B
    uint32_t frame16;    // frame length in copy units (16 B, or 2 B for odd frame sizes)
    uint32_t chunks;     // CTAs per row
    int P, A;
    // sequence minibatches: envs are permuted, not samples; row = t * seq_Be + e holds sample t * N + pi(start + e)
    uint32_t seq_Be;     // 0: flat minibatch
    uint32_t N;
    const uint8_t *done;
    uint8_t *o_done;
};

// One CTA copies one chunk of one row's depth frame with 128-bit loads (no L1 allocation,
// evict-first) and streaming stores; chunk 0 also copies the row's small fields.  VecT is
// uint4 when the frame size is a multiple of 16 bytes, else uint16_t (one fp16 pixel).
template <typename VecT>
__global__ void __launch_bounds__(256) gather_kernel(GatherArgs g, PermParams p) {
    const uint32_t row = blockIdx.x / g.chunks;
    const uint32_t chunk = blockIdx.x - row * g.chunks;
    uint32_t s;
    if (g.seq_Be) {
        const uint32_t t = row / g.seq_Be, e = row - t * g.seq_Be;
        s = t * g.N + perm_apply(p, g.start + e);
    } else {
        s = perm_apply(p, g.start + row);
    }
    const VecT *src = reinterpret_cast<const VecT *>(g.depth) + (size_t)s * g.frame16;
    VecT *dst = reinterpret_cast<VecT *>(g.o_depth) + (size_t)row * g.frame16;
    const uint32_t per = (g.frame16 + g.chunks - 1) / g.chunks;
    const uint32_t lo = chunk * per;
    const uint32_t hi = min(lo + per, g.frame16);
    uint32_t i = lo + threadIdx.x;
    for (; i + 3 * 256 < hi; i += 4 * 256) {
        VecT a = __ldcs(src + i), b = __ldcs(src + i + 256), c = __ldcs(src + i + 512), d = __ldcs(src + i + 768);
        __stcs(dst + i, a);
        __stcs(dst + i + 256, b);
        __stcs(dst + i + 512, c);
        __stcs(dst + i + 768, d);
    }
    for (; i < hi; i += 256) __stcs(dst + i, __ldcs(src + i));
    if (chunk == 0) {
        const int t = threadIdx.x;
        if (t < g.P) g.o_proprio[(size_t)row * g.P + t] = g.proprio[(size_t)s * g.P + t];
        if (t >= 64 && t < 64 + g.A) g.o_action[(size_t)row * g.A + (t - 64)] = g.action[(size_t)s * g.A + (t - 64)];
        if (t == 128) g.o_logp[row] = g.logp[s];
        if (t == 129) g.o_value[row] = g.value[s];
        if (t == 130) g.o_adv[row] = g.adv[s];
        if (t == 131) g.o_ret[row] = g.ret[s];
        if (t == 132 && g.o_index) g.o_index[row] = s;
        if (t == 133 && g.o_done) g.o_done[row] = g.done[s];
    }
}

static int gather_impl(const ppo_buffer *b, uint64_t seed, uint32_t epoch, int mb_index, int num_minibatches,
                       const ppo_minibatch *out, uint8_t *done_out, bool sequences, void *stream);

extern "C" int ppo_shuffle_gather_minibatch(const ppo_buffer *b, uint64_t seed, uint32_t epoch, int mb_index,
                                            int num_minibatches, const ppo_minibatch *out, void *stream) {
    return gather_impl(b, seed, epoch, mb_index, num_minibatches, out, nullptr, false, stream);
}

extern "C" int ppo_shuffle_gather_sequences(const ppo_buffer *b, uint64_t seed, uint32_t epoch, int mb_index,
                                            int num_minibatches, const ppo_minibatch *out, uint8_t *done_out, void *stream) {
    if (!done_out) return PPO_ERR_INVALID_ARG;
    return gather_impl(b, seed, epoch, mb_index, num_minibatches, out, done_out, true, stream);
}

static int gather_impl(const ppo_buffer *b, uint64_t seed, uint32_t epoch, int mb_index, int num_minibatches,
                       const ppo_minibatch *out, uint8_t *done_out, bool sequences, void *stream) {
    if (!b || !out) return PPO_ERR_INVALID_ARG;
    if (num_minibatches <= 0 || mb_index < 0 || mb_index >= num_minibatches) return PPO_ERR_INVALID_ARG;
    // what is permuted and cut into minibatches: the samples, or the envs (each with all its T steps)
    const long long M = sequences ? (long long)b->d.N : (long long)b->d.N * b->d.T;
    if (M % num_minibatches != 0) return PPO_ERR_SHAPE;
    const long long per = M / num_minibatches;
    const long long B = sequences ? per * b->d.T : per;
    if (out->B != B) return PPO_ERR_SHAPE;
    if (!out->depth_f16 || !out->proprio || !out->action || !out->logp_old || !out->value_old || !out->adv ||
        !out->ret)
        return PPO_ERR_INVALID_ARG;
    if (!ppo_aligned(out->depth_f16, 16)) return PPO_ERR_ALIGN;
    if (!b->gae_valid) return PPO_ERR_STATE;
    const size_t frame = (size_t)b->d.H * b->d.W * 2;
    const bool vec16 = frame % 16 == 0;
    if (b->d.P > 64 || b->d.A > 64) return PPO_ERR_UNSUPPORTED;
    GatherArgs g;
    g.depth = b->base + b->field_off[PPO_FIELD_DEPTH];
    g.proprio = slab<float>(b, PPO_FIELD_PROPRIO);
    g.action = slab<float>(b, PPO_FIELD_ACTION);
    g.logp = slab<float>(b, PPO_FIELD_LOGP);
    g.value = slab<float>(b, PPO_FIELD_VALUE);
    g.adv = slab<float>(b, PPO_FIELD_ADV);
    g.ret = slab<float>(b, PPO_FIELD_RET);
    g.o_depth = static_cast<char *>(out->depth_f16);
    g.o_proprio = out->proprio;
    g.o_action = out->action;
    g.o_logp = out->logp_old;
    g.o_value = out->value_old;
    g.o_adv = out->adv;
    g.o_ret = out->ret;
    g.o_index = out->index;
    g.start = (uint32_t)(mb_index * per);
    g.rows = (uint32_t)B;
    g.seq_Be = sequences ? (uint32_t)per : 0u;
    g.N = (uint32_t)b->d.N;
    g.done = slab<uint8_t>(b, PPO_FIELD_DONE);
    g.o_done = done_out;
    g.frame16 = (uint32_t)(vec16 ? frame / 16 : frame / 2);
    // 16 KB per CTA: 4 x 128-bit per thread, so a frame of 38 400 B becomes 3 CTAs
    g.chunks = (uint32_t)((frame + 16383) / 16384);
    g.P = b->d.P;
    g.A = b->d.A;
    const long long ctas = B * g.chunks;
    if (ctas > 0x7fffffffll) return PPO_ERR_UNSUPPORTED;
    PermParams p = make_perm(seed, epoch, (uint32_t)M);
    if (vec16) gather_kernel<uint4><<<(unsigned)ctas, 256, 0, static_cast<cudaStream_t>(stream)>>>(g, p);
    else gather_kernel<uint16_t><<<(unsigned)ctas, 256, 0, static_cast<cudaStream_t>(stream)>>>(g, p);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}
