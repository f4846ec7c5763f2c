// Synthetic depth producer: ray-casts a small analytic scene per env (a plane and a handful of spheres, boxes and
// capsules) straight into slab row t of the rollout buffer's depth field, as fp16.  It stands in for the simulator's
// depth rendering (Section III-C) with plain arithmetic: spatially coherent frames with silhouettes, gradients and
// missing returns instead of noise, produced where the learner reads them.
//
// Camera: pinhole at the origin looking along +z; pixel (v, u) sees the ray through
// ((u + 0.5 - W/2) / f, (v + 0.5 - H/2) / f, 1), f = (W/2) / tan(hfov/2).  With the ray's z component equal to 1 the
// ray parameter of a hit is its depth.  Depths outside [near, far] and rays that hit nothing give 0 (no return).
#include "common.cuh"

namespace {

constexpr int kMaxPrims = 32;
#define kInf __int_as_float(0x7f800000)

__device__ __forceinline__ float hit_sphere(float ox, float oy, float oz, float dx, float dy, float dz, float cx, float cy,
                                            float cz, float r) {
    const float px = ox - cx, py = oy - cy, pz = oz - cz;
    const float a = dx * dx + dy * dy + dz * dz;
    const float b = px * dx + py * dy + pz * dz;
    const float c = px * px + py * py + pz * pz - r * r;
    const float disc = b * b - a * c;
    if (disc < 0.f) return kInf;
    const float s = sqrtf(disc);
    float t = (-b - s) / a;
    if (t > 0.f) return t;
    t = (-b + s) / a;
    return t > 0.f ? t : kInf;
}

__device__ __forceinline__ float hit_box(float dx, float dy, float dz, const float *c, const float *h) {
    const float d[3] = {dx, dy, dz};
    float t0 = 0.f, t1 = kInf;
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        const float lo = c[i] - h[i], hi = c[i] + h[i];
        if (d[i] == 0.f) {
            if (lo > 0.f || hi < 0.f) return kInf;
            continue;
        }
        float a = lo / d[i], b = hi / d[i];
        if (a > b) { const float tmp = a; a = b; b = tmp; }
        t0 = fmaxf(t0, a);
        t1 = fminf(t1, b);
    }
    if (t0 > t1) return kInf;
    return t0 > 0.f ? t0 : ((t1 > 0.f && t1 < kInf) ? t1 : kInf);
}

__device__ __forceinline__ float hit_capsule(float dx, float dy, float dz, const float *pa, const float *ab, float r) {
    float best = hit_sphere(0.f, 0.f, 0.f, dx, dy, dz, pa[0], pa[1], pa[2], r);
    best = fminf(best, hit_sphere(0.f, 0.f, 0.f, dx, dy, dz, pa[0] + ab[0], pa[1] + ab[1], pa[2] + ab[2], r));
    const float l2 = ab[0] * ab[0] + ab[1] * ab[1] + ab[2] * ab[2];
    if (l2 > 0.f) {
        // components of the ray and of the origin perpendicular to the axis
        const float dd = (dx * ab[0] + dy * ab[1] + dz * ab[2]) / l2;
        const float pp = -(pa[0] * ab[0] + pa[1] * ab[1] + pa[2] * ab[2]) / l2;
        const float ex = dx - dd * ab[0], ey = dy - dd * ab[1], ez = dz - dd * ab[2];
        const float qx = -pa[0] - pp * ab[0], qy = -pa[1] - pp * ab[1], qz = -pa[2] - pp * ab[2];
        const float a = ex * ex + ey * ey + ez * ez;
        const float b = qx * ex + qy * ey + qz * ez;
        const float c = qx * qx + qy * qy + qz * qz - r * r;
        const float disc = b * b - a * c;
        if (a > 0.f && disc >= 0.f) {
            const float s = sqrtf(disc);
            const float ts[2] = {(-b - s) / a, (-b + s) / a};
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const float u = pp + ts[k] * dd;
                if (ts[k] > 0.f && u >= 0.f && u <= 1.f) best = fminf(best, ts[k]);
            }
        }
    }
    return best;
}

// One block per (env, 1024-pixel chunk); a thread renders four adjacent pixels and stores them as one 8-byte word.
__global__ void __launch_bounds__(256) depth_render_kernel(__half *__restrict__ depth, int H, int W, float inv_f,
                                                           float near, float far, const float *__restrict__ plane,
                                                           int n_prims, const float *__restrict__ prims, int chunks) {
    __shared__ float sp[kMaxPrims * 8];
    __shared__ float spl[4];
    const int n = blockIdx.x / chunks, chunk = blockIdx.x - n * chunks;
    for (int i = threadIdx.x; i < n_prims * 8; i += 256) sp[i] = prims[(size_t)n * n_prims * 8 + i];
    if (threadIdx.x < 4) spl[threadIdx.x] = plane[(size_t)n * 4 + threadIdx.x];
    __syncthreads();
    const int HW = H * W;
    const int p0 = (chunk * 256 + threadIdx.x) * 4;
    if (p0 >= HW) return;
    __half out[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int p = p0 + j;
        float z = 0.f;
        if (p < HW) {
            const int v = p / W, u = p - v * W;
            const float dx = ((float)u + 0.5f - 0.5f * (float)W) * inv_f, dy = ((float)v + 0.5f - 0.5f * (float)H) * inv_f;
            float best = kInf;
            const float nd = spl[0] * dx + spl[1] * dy + spl[2];
            if (nd != 0.f) {
                const float t = spl[3] / nd;
                if (t > 0.f) best = t;
            }
            for (int k = 0; k < n_prims; ++k) {
                const float *q = sp + k * 8;
                const int type = (int)q[0];
                float t = kInf;
                if (type == 0) t = hit_sphere(0.f, 0.f, 0.f, dx, dy, 1.f, q[1], q[2], q[3], q[4]);
                else if (type == 1) t = hit_box(dx, dy, 1.f, q + 1, q + 4);
                else if (type == 2) t = hit_capsule(dx, dy, 1.f, q + 1, q + 4, q[7]);
                best = fminf(best, t);
            }
            z = (best >= near && best <= far) ? best : 0.f;
        }
        out[j] = __float2half_rn(z);
    }
    __half *dst = depth + (size_t)n * HW + p0;
    if (p0 + 3 < HW && (reinterpret_cast<uintptr_t>(dst) & 7) == 0) {
        *reinterpret_cast<uint2 *>(dst) = *reinterpret_cast<const uint2 *>(out);
    } else {
        for (int j = 0; j < 4 && p0 + j < HW; ++j) dst[j] = out[j];
    }
}

}  // namespace

extern "C" int ppo_buffer_render_depth(ppo_buffer *b, int t, float hfov, float near, float far, const float *plane,
                                       int n_prims, const float *prims, void *stream) {
    if (!b || !plane || (n_prims > 0 && !prims)) return PPO_ERR_INVALID_ARG;
    if (t < 0 || t >= b->d.T || n_prims < 0 || n_prims > kMaxPrims) return PPO_ERR_INVALID_ARG;
    if (!(hfov > 0.f && hfov < 3.14f) || !(near > 0.f) || !(far > near)) return PPO_ERR_INVALID_ARG;
    const ppo_buffer_desc &d = b->d;
    const int HW = d.H * d.W;
    const int chunks = ppo_cdiv(HW, 1024);
    if ((long long)d.N * chunks > 0x7fffffffll) return PPO_ERR_UNSUPPORTED;
    __half *depth = reinterpret_cast<__half *>(b->base + b->field_off[PPO_FIELD_DEPTH]) + (size_t)t * d.N * HW;
    const float inv_f = tanf(0.5f * hfov) / (0.5f * (float)d.W);
    b->gae_valid = false;
    depth_render_kernel<<<(unsigned)(d.N * chunks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        depth, d.H, d.W, inv_f, near, far, plane, n_prims, prims, chunks);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}
