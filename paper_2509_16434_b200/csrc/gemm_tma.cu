// TMA-fed tensor-core versions of the encoder's implicit GEMMs for sm_100a.
//
// One elected thread moves whole operand tiles with cp.async.bulk.tensor (TMA): a box of the NHWC
// activation tensor with a traversal stride of 2 along W and H *is* the im2col tile of one kernel tap
// of a stride-2 convolution, zero padding included (out-of-range parts of a box arrive as zeros), and
// it lands in shared memory already in the swizzled image the UMMA descriptors name.  A second thread
// issues tcgen05.mma into a ring of accumulators in tensor memory; 8 or 16 warps read them back with
// tcgen05.ld for the epilogue.  No thread computes an address per element.
//
//  tma_kmajor_kernel : D[m][n] = sum_k A[m][k] B[n][k], both operands K-major.
//      forward  A = tap boxes of X (row m = output pixel), B = W[co][tap][ci]
//      dgrad    A = shifted boxes of dY (row m = a 2x2 block of input pixels, all four stride-parity classes
//               side by side in the columns), B = the weights regrouped per shift
//  tma_wgrad_kernel  : D[j][co] = sum_m A[m][j] B[m][co], both operands MN-major: the same tap boxes of X
//      and plain boxes of dY, read with the pixel index as the reduction; split over pixel tiles across
//      CTAs, each of which leaves its partial tile in scratch memory; wgrad_reduce_kernel adds the partial
//      tiles to dW in a fixed order, so that the result does not depend on which CTA finishes first.
//
// Tiles follow the pixel grid instead of cutting the flattened pixel index every 128: a tile is a
// rectangle of Wt pixels by R rows of the (image, row) sequence (Wt * R <= 128, chosen to fill most of
// the 128 rows), fetched as one box per image it touches (a tensor map per box height).  A fully
// connected layer is one image with a single row of `batch` pixels, cut into 128-pixel tiles.  Rows of
// the 128-row MMA tile beyond Wt * R are not written and their results are ignored.
//
// Shared-memory rows are 128 bytes (64 channels, SWIZZLE_128B), 64 bytes (32 channels, SWIZZLE_64B) or 32 bytes
// (16 channels, SWIZZLE_32B).
// Every wait is bounded: on a time-out the kernel records PPO_ERR_TIMEOUT, waits (bounded) for the
// copies it has in flight, frees its tensor memory and returns.
#include <cuda.h>  // CUtensorMap and its enums; the encoder is reached through the runtime's entry-point query

#include "gemm.cuh"
#include "tcgen05.cuh"

namespace {

using namespace tc;

constexpr int kMaxTaps = 49;
constexpr int kMaxBoxes = 32;    // boxes per tile; rows per tile are capped at 32 so that this always holds
constexpr int kMaxHeights = 32;  // one tensor map per box height 1 .. 32 rows (a copy costs ~100 cycles to issue,
                                 // so a tile is cut into as few boxes as the image boundaries allow)
constexpr int kMaxStages = 8;
constexpr int kThreads = 192;    // warp 0: TMA producer, warp 1: MMA issue and TMEM owner, warps 2-5: epilogue
constexpr size_t kSmemBudget = 200 * 1024;  // operand stages of the wgrad kernel
constexpr size_t kSmemMax = 227 * 1024;     // dynamic shared memory a CTA may ask for
constexpr size_t kMaxResident = 64 * 1024;

struct Taps {
    int n;
    signed char dy[kMaxTaps], dx[kMaxTaps];
    short wt[kMaxTaps];  // index of the tap inside the weight tensor
};

// Pixel grid the rows of a GEMM walk: Nimg images of Hr rows of Wr pixels.
struct RowGrid {
    int Wr, Hr, Nimg;
    int Wt;     // pixels of a grid row per tile (Wt <= 128)
    int xsegs;  // tiles side by side along a grid row: ceil(Wr / Wt)
    int R;      // grid rows per tile (R * Wt <= 128)
    int tiles;  // tiles over the whole grid: row groups x xsegs
    int arows;  // pixel rows a tile fills in shared memory: R * Wt
};

struct Box {
    int n, y, x;  // image, first row, first pixel
    int hl;       // box height in rows, minus one (index of its tensor map)
    int rowoff;   // first shared-memory row of the box
};

struct Pipe {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint32_t tmem_slot;
    int abort_flag;
    int nboxes;
    Box boxes[kMaxBoxes];
};

// Boxes of the pixel tile whose first grid row is row y of image n and whose first pixel is x0, in
// shared-memory row order.  Rows past the last image get an image index >= Nimg, which the copy engine
// answers with zeros.  Called by one thread.
__host__ __device__ inline int build_boxes_at(const RowGrid &g, int n, int y, int x0, Box *out) {
    int left = g.R, nb = 0, off = 0;
    while (left > 0) {
        int seg = g.Hr - y < left ? g.Hr - y : left;
        left -= seg;
        out[nb++] = {n, y, x0, seg - 1, off};
        y += seg;
        off += seg * g.Wt;
        if (y >= g.Hr) { y = 0; ++n; }
    }
    return nb;
}

// First grid row (image n, row y) and x segment xs of pixel tile mt; advanced tile by tile without divisions
// (a lone thread pays a hundred cycles and more for each).
struct PixTile {
    int mt, xs, n, y;
    __host__ __device__ void init(const RowGrid &g, int mt0) {
        mt = mt0;
        const int rg = mt0 / g.xsegs;
        xs = mt0 - rg * g.xsegs;
        const long long f = (long long)rg * g.R;
        n = (int)(f / g.Hr);
        y = (int)(f - (long long)n * g.Hr);
    }
    __host__ __device__ void advance_to(const RowGrid &g, int target) {
        while (mt < target) {
            ++mt;
            if (++xs == g.xsegs) {
                xs = 0;
                y += g.R;
                while (y >= g.Hr) { y -= g.Hr; ++n; }
            }
        }
    }
};

__host__ __device__ inline int build_boxes(const RowGrid &g, int tile, Box *out) {
    PixTile pt;
    pt.init(g, tile);
    return build_boxes_at(g, pt.n, pt.y, pt.xs * g.Wt, out);
}

// After a time-out: bounded wait for the copies of the last `S` armed stages (iterations it-S .. it-1).
__device__ void drain_copies(uint64_t *full, int it, int S) {
    for (int i = max(0, it - S); i < it; ++i) {
        const long long t0 = clock64();
        while (!mbar_try_wait(&full[i % S], (i / S) & 1))
            if (clock64() - t0 > kWaitCycles / 4) break;
    }
}

// ------------------------------------------------------------------ K-major ----

// Tiles are numbered g = (mt * tiles_n + nt) * ncls + c and every CTA takes one contiguous run of them, so
// that consecutive tiles of a CTA share their pixel tile (the classes of a dgrad) or at least neighbour it.
struct TileCursor {
    int g, g_end, mt, nt, c;
    __device__ void init(int total, int tiles_n, int ncls) {
        const int q = total / (int)gridDim.x, r = total - q * (int)gridDim.x, b = (int)blockIdx.x;
        g = b * q + (b < r ? b : r);
        g_end = g + q + (b < r ? 1 : 0);
        c = g % ncls;
        const int t = g / ncls;
        nt = t % tiles_n;
        mt = t / tiles_n;
    }
    __device__ bool valid() const { return g < g_end; }
    __device__ void next(int tiles_n, int ncls) {
        ++g;
        if (++c == ncls) {
            c = 0;
            if (++nt == tiles_n) { nt = 0; ++mt; }
        }
    }
};

// One group of output columns with its own tap list: the whole GEMM for a forward pass; for a merged dgrad
// one tile of BN columns of the (parity class, input channel) axis, which only some shifts reach.
struct KClass {
    int b_row0;  // first weight row (output column) of the group
    Taps taps;
};

enum { EPI_FWD = 0, EPI_HEAD = 1, EPI_DGRAD = 2 };

constexpr int kEpiWarps = 16;                     // at most: two or four warps per TMEM lane quarter share out the column groups
constexpr int kKThreads = (2 + kEpiWarps) * 32;   // warp 0: TMA producer, warp 1: MMA issue and TMEM owner
constexpr int kMaxBias = 512;
constexpr int kMaxWtab = 64;

// A pipeline stage carries G sub-blocks; sub-block q of a tile is (tap, channel chunk) = divmod(q, kchunks):
// the A boxes of that tap (128 rows) followed, unless the weights are resident, by its BN weight rows.
struct KArgs {
    CUtensorMap mapA[kMaxHeights];
    CUtensorMap mapB;
    RowGrid grid;
    int s_mul, s_oy, s_ox;  // source pixel of tap t: (y * s_mul + s_oy + dy[t], x * s_mul + s_ox + dx[t])
    int CB, row_bytes;      // channels per box (64, 32 or 16) and bytes of a shared-memory row
    int kchunks;            // boxes along the channels of one tap
    int w_tap;              // elements between taps in a weight row
    int G, nbmax;           // sub-blocks per stage; most A boxes a tile has
    int tmem_cap;           // tensor-memory columns this CTA may take: 512, or 256 when two CTAs share an SM
    int nepi;               // epilogue warps: 8, or 16 where the epilogue is the heavier side (dgrad with gate bits)
    int wres, wtaps;        // weights resident in shared memory (all wtaps * kchunks boxes, loaded once)
    int N, BN, tiles_n, total_tiles, ncls, stages;  // tile g = ((mt * tiles_n) + nt) * ncls + class
    int Hout, Wout, ldo;
    int nq_ci;  // merged dgrad: channels per parity class (column n = class * nq_ci + channel), else 0
    long long cls_orows;  // output rows between the classes' results (split reduction of a flat GEMM), else 0
    int mode, relu, A;
    const float *bias;
    bf16 *out;
    float *out_f32;
    const bf16 *mask;
    const uint32_t *mask_bits;  // merged dgrad: the gate as bits, [pixels][nq_ci / 32]
    uint32_t *out_bits;         // forward: gate bits of the ReLU output, [pixels][N / 32]
    float *mean, *value;
    const float *ln_gamma, *ln_beta;  // forward with layer normalisation over the N columns of a row (null: none)
    bf16 *ln_xhat;
    float *ln_rstd;
    int32_t *status;
    KClass cls[4];
};

struct PipeK {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tfull[4];
    uint64_t tempty[4];
    uint64_t wfull;
    uint32_t tmem_slot;
    int abort_flag;
    int nboxes;
    Box boxes[kMaxBoxes];
    uint32_t wtab[4][kMaxWtab];  // resident weights: (byte offset >> 4) of the box that sub-block q of a class reads
    alignas(16) float bias[kMaxBias];
    alignas(16) float gamma[256], beta[256];  // layer normalisation (N <= 256)
    // followed by the epilogue staging: per epilogue warp 32 rows x 32 bf16 columns (2 KB), 16-byte pieces swizzled
};

__global__ void __launch_bounds__(kKThreads, 1) tma_kmajor_kernel(const __grid_constant__ KArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int BN = a.BN, S = a.stages, G = a.G;
    const uint32_t rb = (uint32_t)a.row_bytes;
    const uint32_t a_bytes = 128u * rb, b_bytes = (uint32_t)BN * rb;
    const uint32_t sub_bytes = a_bytes + (a.wres ? 0u : b_bytes);
    const uint32_t stage_bytes = (uint32_t)G * sub_bytes;
    const uint32_t res_bytes = a.wres ? (uint32_t)(a.wtaps * a.kchunks) * b_bytes : 0u;
    PipeK *pipe = reinterpret_cast<PipeK *>(smem + (size_t)S * stage_bytes + res_bytes);
    volatile int *abort_flag = &pipe->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // ring of accumulators in tensor memory: four when they fit in its 512 columns, else two
    const uint32_t acc_cols = tmem_cols_for(BN);
    const int nacc_log = acc_cols * 4 <= (uint32_t)a.tmem_cap ? 2 : 1, nacc = 1 << nacc_log;
    const uint32_t ncols = acc_cols * nacc;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe->full[s], 1);
            mbar_init(&pipe->empty[s], 1);
        }
        for (int i = 0; i < nacc; ++i) {
            mbar_init(&pipe->tfull[i], 1);
            mbar_init(&pipe->tempty[i], a.nepi * 32);
        }
        mbar_init(&pipe->wfull, 1);
        pipe->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (a.mode != EPI_DGRAD)
        for (int i = threadIdx.x; i < a.tiles_n * BN; i += (int)blockDim.x) pipe->bias[i] = i < a.N ? a.bias[i] : 0.f;
    if (a.ln_gamma)
        for (int i = threadIdx.x; i < 256; i += (int)blockDim.x) {
            pipe->gamma[i] = i < a.N ? a.ln_gamma[i] : 0.f;
            pipe->beta[i] = i < a.N ? a.ln_beta[i] : 0.f;
        }
    if (a.wres)
        for (int i = threadIdx.x; i < a.ncls * kMaxWtab; i += (int)blockDim.x) {
            const int c = i / kMaxWtab, q = i - c * kMaxWtab;
            const int tap = q / a.kchunks, kc = q - tap * a.kchunks;
            if (tap < a.cls[c].taps.n)
                pipe->wtab[c][q] = (uint32_t)((int)a.cls[c].taps.wt[tap] * a.kchunks + kc) * (b_bytes >> 4);
        }
    if (warp == 1) tmem_alloc(&pipe->tmem_slot, ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = pipe->tmem_slot;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t res_base = smem_base + (uint32_t)S * stage_bytes;

    if (warp == 0) {
        // ---------------- TMA producer: the lanes share out the copies of a stage, one thread each
        if (a.wres) {
            const int nw = a.wtaps * a.kchunks;
            if (lane == 0) mbar_arrive_expect_tx(&pipe->wfull, (uint32_t)nw * b_bytes);
            __syncwarp();
            for (int q = lane; q < nw; q += 32) {
                const int tap = q / a.kchunks, kc = q - tap * a.kchunks;
                tma_load_2d(res_base + (uint32_t)q * b_bytes, &a.mapB, &pipe->wfull, tap * a.w_tap + kc * a.CB, 0);
            }
        }
        // Lane l owns copy j = l % lps of sub-block slot gi = l / lps of every stage (G * lps <= 32): its
        // A box of the tile, or the weight rows.  Per stage a lane only advances (tap, chunk) and issues.
        const int lps = a.nbmax + (a.wres ? 0 : 1);
        const int gi = lane / lps, j = lane - gi * lps;
        const bool lane_on = gi < G;
        const bool is_b = !a.wres && j == a.nbmax;
        const uint32_t tx_sub = (uint32_t)a.grid.arows * rb + (a.wres ? 0u : b_bytes);
        int it = 0, s = 0;
        uint32_t ph = 0;
        bool ok = true;
        TileCursor tc_;
        tc_.init(a.total_tiles, a.tiles_n, a.ncls);
        PixTile pt;
        pt.init(a.grid, tc_.mt);
        int last_mt = -1;
        bool have = false;
        Box bx = {0, 0, 0, 0, 0};
        const int tap0 = gi / a.kchunks, kc0 = gi - tap0 * a.kchunks;
        for (; tc_.valid() && ok; tc_.next(a.tiles_n, a.ncls)) {
            const int n0 = tc_.nt * BN;
            const KClass &k = a.cls[tc_.c];
            if (tc_.mt != last_mt) {
                last_mt = tc_.mt;
                pt.advance_to(a.grid, tc_.mt);
                if (lane == 0) pipe->nboxes = build_boxes_at(a.grid, pt.n, pt.y, pt.xs * a.grid.Wt, pipe->boxes);
                __syncwarp();
                have = lane_on && (is_b || j < pipe->nboxes);
                if (have && !is_b) bx = pipe->boxes[j];
                __syncwarp();
            }
            const uint32_t dst_off = (uint32_t)gi * sub_bytes + (is_b ? a_bytes : (uint32_t)bx.rowoff * rb);
            const int cx = bx.x * a.s_mul + a.s_ox, cy = bx.y * a.s_mul + a.s_oy;
            const void *map = is_b ? (const void *)&a.mapB : (const void *)&a.mapA[bx.hl];
            const int ntaps = k.taps.n, nsub = ntaps * a.kchunks;
            int tap = tap0, kc = kc0;
            for (int q0 = 0; q0 < nsub; q0 += G, ++it) {
                int okw = 1;
                if (lane == 0) okw = mbar_wait(&pipe->empty[s], ph ^ 1u, abort_flag, a.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, okw, 0) != 0;
                if (!ok) break;
                if (lane == 0) mbar_arrive_expect_tx(&pipe->full[s], (uint32_t)min(G, nsub - q0) * tx_sub);
                __syncwarp();
                if (have && tap < ntaps) {
                    const uint32_t dst = smem_base + (uint32_t)s * stage_bytes + dst_off;
                    if (is_b) tma_load_2d(dst, map, &pipe->full[s], (int)k.taps.wt[tap] * a.w_tap + kc * a.CB, n0 + k.b_row0);
                    else tma_load_4d(dst, map, &pipe->full[s], kc * a.CB, cx + k.taps.dx[tap], cy + k.taps.dy[tap], bx.n);
                }
                kc += G;
                while (kc >= a.kchunks) { kc -= a.kchunks; ++tap; }
                if (++s == S) { s = 0; ph ^= 1u; }
            }
        }
        if (!ok && lane == 0) drain_copies(pipe->full, it, S);
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issue: one thread feeds the tensor core.  Its instruction stream is the
        // ceiling of the whole kernel (a lone thread issues a dependent instruction only every few cycles),
        // so the descriptors are built once and advanced by adds.
        const uint32_t idesc = instr_desc(128, BN, 0, 0);
        const uint32_t sbo = 8u * rb;
        const uint64_t d0 = smem_desc_sw(smem_base, 16, sbo, rb);
        const uint32_t d_lo0 = (uint32_t)d0, d_hi = (uint32_t)(d0 >> 32);
        const uint32_t res_lo0 = d_lo0 + ((res_base - smem_base) >> 4);
        const uint32_t stage16 = stage_bytes >> 4, sub16 = sub_bytes >> 4, ab16 = a_bytes >> 4;
        const int ksteps = a.CB >> 4;  // 4, 2 or 1 K = 16 steps per box (32 bytes each along the swizzled row)
        int ti = 0, s = 0;
        uint32_t ph = 0;
        bool ok = true;
        if (a.wres) ok = mbar_wait(&pipe->wfull, 0, abort_flag, a.status);
        TileCursor tc_;
        for (tc_.init(a.total_tiles, a.tiles_n, a.ncls); tc_.valid() && ok; tc_.next(a.tiles_n, a.ncls), ++ti) {
            const int c = tc_.c;
            const int nsub = a.cls[c].taps.n * a.kchunks;
            const uint32_t *tbl = pipe->wtab[c];
            const int acc = ti & (nacc - 1);
            ok = mbar_wait(&pipe->tempty[acc], ((ti >> nacc_log) & 1) ^ 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t tmem_d = tmem_base + acc * acc_cols;
            uint32_t accum = 0;
            for (int q0 = 0; q0 < nsub; q0 += G) {
                ok = mbar_wait(&pipe->full[s], ph, abort_flag, a.status);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const int nval = min(G, nsub - q0);
                    uint32_t la = d_lo0 + (uint32_t)s * stage16;
                    for (int gi = 0; gi < nval; ++gi, la += sub16) {
                        const uint32_t lb = a.wres ? res_lo0 + tbl[q0 + gi] : la + ab16;
                        umma_bf16_lh(tmem_d, la, d_hi, lb, d_hi, idesc, accum);
                        if (ksteps >= 2) umma_bf16_lh(tmem_d, la + 2, d_hi, lb + 2, d_hi, idesc, 1u);
                        if (ksteps == 4) {
                            umma_bf16_lh(tmem_d, la + 4, d_hi, lb + 4, d_hi, idesc, 1u);
                            umma_bf16_lh(tmem_d, la + 6, d_hi, lb + 6, d_hi, idesc, 1u);
                        }
                        accum = 1u;
                    }
                    umma_commit(&pipe->empty[s]);
                }
                __syncwarp();
                if (++s == S) { s = 0; ph ^= 1u; }
            }
            if (ok && lane == 0) umma_commit(&pipe->tfull[acc]);
            __syncwarp();
        }
    } else {
        // ---------------- epilogue: warp w reads TMEM lanes 32 (w % 4) .. +31; the two warps of a lane
        // quarter take alternate 16-column chunks
        const int lg = warp & 3, ew4 = (warp - 2) >> 2, wq = a.nepi >> 2;  // ew4: which of the quarter's wq warps
        const int p = lg * 32 + lane;
        const RowGrid &gr = a.grid;
        int ti = 0;
        bool ok = true;
        TileCursor tc_;
        tc_.init(a.total_tiles, a.tiles_n, a.ncls);
        PixTile pt;
        pt.init(gr, tc_.mt);
        int last_mt = -1;
        bool pix_ok = false;  // tile row p is a pixel of the grid
        int n = 0, y = 0, x = 0;
        const int fr = p / gr.Wt, xx = p - fr * gr.Wt;  // row and pixel of tile row p inside the tile rectangle
        for (; tc_.valid() && ok; tc_.next(a.tiles_n, a.ncls), ++ti) {
            const int n0 = tc_.nt * BN;
            const KClass &k = a.cls[tc_.c];
            if (tc_.mt != last_mt) {  // pixel of tile row p
                last_mt = tc_.mt;
                pt.advance_to(gr, tc_.mt);
                x = pt.xs * gr.Wt + xx;
                n = pt.n;
                y = pt.y + fr;
                while (y >= gr.Hr) { y -= gr.Hr; ++n; }
                pix_ok = fr < gr.R && x < gr.Wr && n < gr.Nimg;
            }
            // Output row and column of this thread's accumulator columns c0 .. c0+15.  Forward and flat GEMMs:
            // the pixel itself.  Merged dgrad: column class * nq_ci + channel belongs to input pixel
            // (2y + class / 2, 2x + class % 2).
            auto locate = [&](int c0, long long &orow, int &col) -> bool {
                col = n0 + c0;
                int oy = y, ox = x;
                if (a.nq_ci) {
                    const int gc = k.b_row0 + col, q = gc / a.nq_ci;
                    col = gc - q * a.nq_ci;
                    oy = 2 * y + (q >> 1);
                    ox = 2 * x + (q & 1);
                }
                orow = ((long long)n * a.Hout + oy) * a.Wout + ox + tc_.c * a.cls_orows;
                return pix_ok && oy < a.Hout && ox < a.Wout;
            };
            const int ncol = a.nq_ci ? a.nq_ci : a.N;  // columns of an output row
            const bool use_bits = a.mode == EPI_DGRAD && a.mask_bits != nullptr;
            const bool use_mask = a.mode == EPI_DGRAD && a.mask != nullptr && !use_bits;
            const int acc = ti & (nacc - 1);
            const uint32_t lane_base = tmem_base + acc * acc_cols + ((uint32_t)(lg * 32) << 16);
            if (a.out != nullptr && a.out_f32 == nullptr && a.mode != EPI_HEAD && !use_mask) {
                // ---- bf16 outputs, staged: a thread owns a pixel (its TMEM lane), but a warp that stores 32
                // pixels with one instruction touches 32 cache lines.  So 32-column groups pass through a small
                // swizzled shared-memory tile: four lanes then move one pixel's 64 contiguous bytes, and an
                // instruction covers 8 lines.  The ReLU mask comes in the same way, and the first group's mask
                // is fetched before the accumulator is waited for, so that its latency overlaps the MMAs.
                uint4 *stg = reinterpret_cast<uint4 *>(pipe + 1) + (size_t)(warp - 2) * 128;
                const int sw = (lane >> 1) & 3;
                const int rr0 = lane >> 2, piece = lane & 3;
                // this warp's groups: columns (ew4 + wq g) * 32; at most 4 (BN <= 256, wq >= 2)
                int ng = 0;
                for (int c0 = ew4 * 32; c0 < BN && n0 + c0 < a.N; c0 += wq * 32) ++ng;
                uint32_t gbits[4] = {0u, 0u, 0u, 0u};
                if (use_bits) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (g < ng) {
                            long long orow;
                            int col;
                            if (locate((ew4 + wq * g) * 32, orow, col)) gbits[g] = a.mask_bits[orow * (ncol >> 5) + (col >> 5)];
                        }
                    }
                }
                ok = mbar_wait(&pipe->tfull[acc], (ti >> nacc_log) & 1, abort_flag, a.status);
                if (!ok) break;
                tc_fence_after();
                // Layer normalisation: this thread's row holds all N channels of its pixel in the accumulator, so
                // every warp of the lane quarter walks the whole row twice (mean, then variance about it) before it
                // normalises its own column groups.
                float ln_mean = 0.f, ln_rs = 0.f;
                if (a.ln_gamma) {
                    float sum = 0.f;
                    for (int c0 = 0; c0 < a.N; c0 += 16) {
                        float t[16];
                        tmem_ld16(lane_base + (uint32_t)c0, t);
#pragma unroll
                        for (int i = 0; i < 16; ++i) sum += t[i] + pipe->bias[c0 + i];
                    }
                    ln_mean = sum / (float)a.N;
                    float sq = 0.f;
                    for (int c0 = 0; c0 < a.N; c0 += 16) {
                        float t[16];
                        tmem_ld16(lane_base + (uint32_t)c0, t);
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const float dlt = t[i] + pipe->bias[c0 + i] - ln_mean;
                            sq += dlt * dlt;
                        }
                    }
                    ln_rs = rsqrtf(sq / (float)a.N + kLnEps);
                }
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (g >= ng) break;
                    const int c0 = (ew4 + wq * g) * 32;
                    float v[32];
                    tmem_ld16(lane_base + (uint32_t)c0, v);
                    if (c0 + 16 < BN) tmem_ld16(lane_base + (uint32_t)c0 + 16u, v + 16);
                    long long orow;
                    int col;
                    const int okr = locate(c0, orow, col) ? 1 : 0;
                    uint32_t pk[16];
                    if (a.mode == EPI_FWD) {
                        const float4 *bp = reinterpret_cast<const float4 *>(pipe->bias + n0 + c0);
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const float4 bv = bp[q];
                            v[4 * q] += bv.x; v[4 * q + 1] += bv.y; v[4 * q + 2] += bv.z; v[4 * q + 3] += bv.w;
                        }
                        if (a.ln_gamma) {
                            // the normalised values go out first (same staging, same store pattern), then v becomes
                            // gamma * xhat + beta and takes the usual path
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = (v[i] - ln_mean) * ln_rs;
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                stg[lane * 4 + (j ^ sw)] = make_uint4(pack_bf16x2(v[8 * j], v[8 * j + 1]), pack_bf16x2(v[8 * j + 2], v[8 * j + 3]),
                                                                       pack_bf16x2(v[8 * j + 4], v[8 * j + 5]), pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
                            __syncwarp();
#pragma unroll
                            for (int ps = 0; ps < 4; ++ps) {
                                const int rr = ps * 8 + rr0;
                                const long long o_r = __shfl_sync(0xffffffffu, orow, rr);
                                const int ok_r = __shfl_sync(0xffffffffu, okr, rr);
                                if (ok_r && col + piece * 8 < ncol && c0 + piece * 8 < BN)
                                    *reinterpret_cast<uint4 *>(a.ln_xhat + o_r * a.ldo + col + piece * 8) =
                                        stg[rr * 4 + (piece ^ ((rr >> 1) & 3))];
                            }
                            __syncwarp();
                            if (okr && c0 == 0) a.ln_rstd[orow] = ln_rs;
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = fmaf(pipe->gamma[c0 + i], v[i], pipe->beta[c0 + i]);
                        }
                        if (a.relu) {
                            uint32_t w = 0;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                pk[j] = relu_pack_bf16x2(v[2 * j], v[2 * j + 1]);
                                w = gate_bits_add(w, pk[j], j);
                            }
                            if (a.out_bits && okr) a.out_bits[orow * (a.N >> 5) + (col >> 5)] = w;
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(v[2 * j], v[2 * j + 1]);
                        }
                    } else if (use_bits) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(v[2 * j], v[2 * j + 1]) & gate_pair_mask(gbits[g], j);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(v[2 * j], v[2 * j + 1]);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        stg[lane * 4 + (j ^ sw)] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                    __syncwarp();
#pragma unroll
                    for (int ps = 0; ps < 4; ++ps) {
                        const int rr = ps * 8 + rr0;
                        const long long o_r = __shfl_sync(0xffffffffu, orow, rr);
                        const int ok_r = __shfl_sync(0xffffffffu, okr, rr);
                        if (ok_r && col + piece * 8 < ncol && c0 + piece * 8 < BN)
                            *reinterpret_cast<uint4 *>(a.out + o_r * a.ldo + col + piece * 8) =
                                stg[rr * 4 + (piece ^ ((rr >> 1) & 3))];
                    }
                    __syncwarp();
                }
                tc_fence_before();
                mbar_arrive(&pipe->tempty[acc]);
                continue;
            }
            // ---- head and fp32 outputs (small): every thread stores its own row
            ok = mbar_wait(&pipe->tfull[acc], (ti >> nacc_log) & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            for (int c0 = ew4 * 16; c0 < BN; c0 += wq * 16) {
                if (n0 + c0 >= a.N) break;  // uniform across the warp
                float v[16];
                tmem_ld16(lane_base + (uint32_t)c0, v);
                long long orow;
                int nn;
                if (!locate(c0, orow, nn)) continue;
                if (a.mode == EPI_HEAD) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        if (nn + i < a.A) a.mean[orow * a.A + nn + i] = v[i] + pipe->bias[nn + i];
                        else if (nn + i == a.A) a.value[orow] = v[i] + pipe->bias[nn + i];
                    }
                    continue;
                }
                if (use_mask) {
                    const uint4 *mp = reinterpret_cast<const uint4 *>(a.mask + orow * a.ldo + nn);
#pragma unroll
                    for (int hlf = 0; hlf < 2; ++hlf) {
                        if (nn + hlf * 8 < ncol) {
                            const uint4 mk = mp[hlf];
                            const __nv_bfloat162 *m2 = reinterpret_cast<const __nv_bfloat162 *>(&mk);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 f = __bfloat1622float2(m2[i]);
                                if (!(f.x > 0.f)) v[hlf * 8 + 2 * i] = 0.f;
                                if (!(f.y > 0.f)) v[hlf * 8 + 2 * i + 1] = 0.f;
                            }
                        }
                    }
                }
                if (a.out) {
                    uint4 *op = reinterpret_cast<uint4 *>(a.out + orow * a.ldo + nn);
#pragma unroll
                    for (int hlf = 0; hlf < 2; ++hlf) {
                        if (nn + hlf * 8 < ncol) {
                            __nv_bfloat162 pk[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                pk[i] = __floats2bfloat162_rn(v[hlf * 8 + 2 * i], v[hlf * 8 + 2 * i + 1]);
                            op[hlf] = *reinterpret_cast<uint4 *>(pk);
                        }
                    }
                }
                if (a.out_f32) {
                    float4 *op = reinterpret_cast<float4 *>(a.out_f32 + orow * a.ldo + nn);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (nn + q * 4 < ncol) op[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                }
            }
            tc_fence_before();
            mbar_arrive(&pipe->tempty[acc]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, ncols);
    }
}

// -------------------------------------------------------------------- wgrad ----

struct WArgs {
    CUtensorMap mapA[kMaxHeights];  // tap boxes of X (traversal stride 2 for a convolution)
    CUtensorMap mapB[kMaxHeights];  // boxes of dY over the same pixels
    RowGrid grid;                   // output pixels
    int s_mul, pad, ksz, ntaps;
    int CB, rbA, mblocks, kchunks;  // A: channels per box, row bytes, boxes per 128 columns, boxes per tap
    int CBn, rbB, nblocks, BN;      // B: likewise over the output channels of this tile
    int Kfwd, Co;
    int tiles_per_split, nmma, stages;
    float *part;                    // partial tiles [split][column tile][row tile][BN][128] fp32
    // Bias gradient db[co] += sum over pixels of dY, or null.  The last column tile has an A block that no tap
    // fills; its first column is set to ones, so row ones_blk * CB of that tile's accumulator is the column
    // sum of dY: the pass over dY that a separate reduction kernel would make comes for free.
    int has_db;
    int ones_blk;
    int32_t *status;
};

__global__ void __launch_bounds__(kThreads, 1) tma_wgrad_kernel(const __grid_constant__ WArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int BN = a.BN, S = a.stages;
    const uint32_t rbA = (uint32_t)a.rbA, rbB = (uint32_t)a.rbB;
    const uint32_t a_bytes = 128u * 256u;                 // 128 pixel rows x 128 columns of bf16
    const uint32_t stage_bytes = a_bytes + 128u * 2u * (uint32_t)BN;
    Pipe *pipe = reinterpret_cast<Pipe *>(smem + (size_t)S * stage_bytes);
    volatile int *abort_flag = &pipe->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ncols = tmem_cols_for(BN);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe->full[s], 1);
            mbar_init(&pipe->empty[s], 1);
        }
        mbar_init(&pipe->tfull[0], 1);
        pipe->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Rows and column blocks no copy ever writes must read as zeros: the pixel index is the reduction.
    {
        uint4 *z = reinterpret_cast<uint4 *>(smem);
        const uint32_t n16 = (uint32_t)S * stage_bytes / 16u;
        for (uint32_t i = threadIdx.x; i < n16; i += kThreads) z[i] = make_uint4(0, 0, 0, 0);
    }
    const bool ones_tile = a.has_db && blockIdx.x == gridDim.x - 1;
    if (ones_tile) {
        // channel 0 of block ones_blk, all 128 pixel rows of every stage: the first element of 16-byte piece 0,
        // which the swizzle moves to piece (row & 7) of a 128-byte row, ((row >> 1) & 3) of a 64-byte row,
        // ((row >> 2) & 1) of a 32-byte row
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < (uint32_t)S * 128u; i += kThreads) {
            const uint32_t s = i >> 7, r = i & 127u;
            const uint32_t piece = rbA == 128u ? (r & 7u) : (rbA == 64u ? ((r >> 1) & 3u) : ((r >> 2) & 1u));
            *reinterpret_cast<bf16 *>(smem + (size_t)s * stage_bytes + (size_t)a.ones_blk * 128u * rbA + r * rbA + piece * 16u) =
                __float2bfloat16_rn(1.f);
        }
    }
    fence_async_smem();
    if (warp == 1) tmem_alloc(&pipe->tmem_slot, ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = pipe->tmem_slot;
    const uint32_t smem_base = smem_u32(smem);

    const int jb0 = blockIdx.x * a.mblocks;  // first (tap, channel chunk) box of this column tile
    const int co0 = blockIdx.y * BN;
    const int t_lo = blockIdx.z * a.tiles_per_split;
    const int t_hi = min(a.grid.tiles, t_lo + a.tiles_per_split);
    const int nkb = max(0, t_hi - t_lo);
    int nvalid = 0;
    for (int i = 0; i < a.mblocks; ++i)
        if ((jb0 + i) / a.kchunks < a.ntaps) ++nvalid;
    const uint32_t tx_bytes = (uint32_t)a.grid.arows * ((uint32_t)nvalid * rbA + (uint32_t)a.nblocks * rbB);

    if (warp == 0) {
        // ---------------- TMA producer: the lanes share out the copies of a K block, one thread each
        // Lane l owns copy i = l % per_box (an A column block, then the B blocks) of box l / per_box of every
        // pixel tile; tiles with more boxes than that go round again.
        const int per_box = nvalid + a.nblocks;
        const int b_l = lane / per_box, i_l = lane - b_l * per_box;
        const int boxes_per_round = 32 / per_box;
        int tap = 0, kc = 0, kh = 0, kw = 0;
        if (i_l < nvalid) {
            const int jb = jb0 + i_l;
            tap = jb / a.kchunks;
            kc = jb - tap * a.kchunks;
            kh = tap / a.ksz;
            kw = tap - kh * a.ksz;
        }
        const bool is_a = i_l < nvalid;
        const uint32_t rbu = is_a ? rbA : rbB;
        const uint32_t blk_off = is_a ? (uint32_t)i_l * 128u * rbA : a_bytes + (uint32_t)(i_l - nvalid) * 128u * rbB;
        const int c0 = is_a ? kc * a.CB : co0 + (i_l - nvalid) * a.CBn;
        const int mul = is_a ? a.s_mul : 1, ox = is_a ? kw - a.pad : 0, oy = is_a ? kh - a.pad : 0;
        const CUtensorMap *maps = is_a ? a.mapA : a.mapB;
        bool ok = true;
        int kb = 0, s = 0;
        uint32_t ph = 0;
        PixTile pt;
        pt.init(a.grid, t_lo);
        for (; kb < nkb; ++kb) {
            int okw = 1;
            if (lane == 0) okw = mbar_wait(&pipe->empty[s], ph ^ 1u, abort_flag, a.status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, okw, 0) != 0;
            if (!ok) break;
            if (lane == 0) {
                mbar_arrive_expect_tx(&pipe->full[s], tx_bytes);
                pt.advance_to(a.grid, t_lo + kb);
                pipe->nboxes = build_boxes_at(a.grid, pt.n, pt.y, pt.xs * a.grid.Wt, pipe->boxes);
            }
            __syncwarp();
            const int nb = pipe->nboxes;
            const uint32_t st = smem_base + (uint32_t)s * stage_bytes + blk_off;
            if (b_l < boxes_per_round)
                for (int b = b_l; b < nb; b += boxes_per_round) {
                    const Box bx = pipe->boxes[b];
                    tma_load_4d(st + (uint32_t)bx.rowoff * rbu, &maps[bx.hl], &pipe->full[s], c0, bx.x * mul + ox,
                                bx.y * mul + oy, bx.n);
                }
            __syncwarp();
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (!ok && lane == 0) drain_copies(pipe->full, kb, S);
        __syncwarp();
    } else if (warp == 1) {
        const uint32_t idesc = instr_desc(128, BN, 1, 1);
        const uint64_t dA = smem_desc_sw(smem_base, 128u * rbA, 8u * rbA, rbA);
        const uint64_t dB = smem_desc_sw(smem_base + a_bytes, 128u * rbB, 8u * rbB, rbB);
        const uint32_t a_hi = (uint32_t)(dA >> 32), b_hi = (uint32_t)(dB >> 32);
        const uint32_t stepA = rbA, stepB = rbB;  // 16 pixel rows per instruction: (16 * row bytes) >> 4
        bool ok = true;
        uint32_t accum = 0, ph = 0;
        int s = 0;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            ok = mbar_wait(&pipe->full[s], ph, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                uint32_t la = (uint32_t)dA + (uint32_t)s * (stage_bytes >> 4), lb = (uint32_t)dB + (uint32_t)s * (stage_bytes >> 4);
                for (int k = 0; k < a.nmma; ++k, la += stepA, lb += stepB) {
                    umma_bf16_lh(tmem_d, la, a_hi, lb, b_hi, idesc, accum);
                    accum = 1u;
                }
                umma_commit(&pipe->empty[s]);
            }
            __syncwarp();
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (ok && nkb > 0 && lane == 0) umma_commit(&pipe->tfull[0]);
        __syncwarp();
    } else if (nkb > 0) {
        // ---------------- epilogue: TMEM lane p is row p of this CTA's 128 x BN tile of dW^T; the whole tile goes
        // to the CTA's slot of the scratch array, column by column (a warp's store covers 32 consecutive rows)
        const int lg = warp & 3;
        const int p = lg * 32 + lane;
        if (mbar_wait(&pipe->tfull[0], 0, abort_flag, a.status)) {
            tc_fence_after();
            float *tile = a.part + ((size_t)(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * (size_t)(128 * BN);
            const uint32_t lane_base = tmem_d + ((uint32_t)(lg * 32) << 16);
            for (int c0 = 0; c0 < BN; c0 += 16) {
                float v[16];
                tmem_ld16(lane_base + (uint32_t)c0, v);
#pragma unroll
                for (int i = 0; i < 16; ++i) tile[(c0 + i) * 128 + p] = v[i];
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, ncols);
    }
}

// dW[co][jj] += sum over the splits, in their order, of the partial tiles a split-K weight-gradient kernel left
// in `part` ([split][column tile y][row tile x][BN][128]); threads past Co * Kfwd do the same for the bias gradient,
// whose partial sums sit in row `ones_row` of dW^T (db == null: there is none).
__global__ void __launch_bounds__(256) wgrad_reduce_kernel(const float *__restrict__ part, int jtiles, int ctiles,
                                                           int splits, int BN, int Kfwd, int Co, float *__restrict__ dW,
                                                           float *__restrict__ db, int ones_row) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nW = (long long)Co * Kfwd;
    int co, jj;
    float *dst;
    if (idx < nW) {
        co = (int)(idx / Kfwd);
        jj = (int)(idx - (long long)co * Kfwd);
        dst = dW + idx;
    } else if (db != nullptr && idx < nW + Co) {
        co = (int)(idx - nW);
        jj = ones_row;
        dst = db + co;
    } else {
        return;
    }
    const int x = jj >> 7, p = jj & 127, y = co / BN, c = co - y * BN;
    const size_t tile = (size_t)128 * BN, per_split = (size_t)ctiles * jtiles * tile;
    const float *src = part + ((size_t)y * jtiles + x) * tile + (size_t)c * 128 + p;
    float acc = 0.f;
    for (int z = 0; z < splits; ++z) acc += src[(size_t)z * per_split];
    *dst += acc;
}

// --------------------------------------------------------------------- host ----

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Map of a bf16 tensor [d3][d2][d1][d0] whose innermost rows are `ld` elements apart; box and traversal
// strides innermost first.  `row_bytes` selects the swizzle (box[0] * 2 == row_bytes).
int make_map(CUtensorMap *m, const void *base, int rank, const long long *dims, long long ld, const int *box,
             const int *estride, int row_bytes) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return PPO_ERR_CUDA;
    cuuint64_t gd[4];
    cuuint64_t gs[3];
    cuuint32_t bx[4], es[4];
    for (int i = 0; i < rank; ++i) {
        gd[i] = (cuuint64_t)dims[i];
        bx[i] = (cuuint32_t)box[i];
        es[i] = (cuuint32_t)estride[i];
        if (box[i] < 1 || box[i] > 256 || dims[i] < 1) return PPO_ERR_UNSUPPORTED;
    }
    long long s = ld * 2;
    for (int i = 0; i + 1 < rank; ++i) {
        if (s % 16 != 0 || s >= (1ll << 40)) return PPO_ERR_UNSUPPORTED;
        gs[i] = (cuuint64_t)s;
        s *= dims[i + 1];
    }
    if (box[0] * 2 != row_bytes || !ppo_aligned(base, 16)) return PPO_ERR_UNSUPPORTED;
    const CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), gd, gs, bx,
                          es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PPO_OK : PPO_ERR_CUDA;
}

// Channels per box for a source of C channels per pixel (`flat`: a 1x1 image, where a ragged last box is
// completed with zeros by the copy engine), or 0 when the TMA kernels do not cover it.
int channels_per_box(int C, bool flat) {
    if (C % 64 == 0) return 64;
    if (flat) return (C >= 64 && C % 8 == 0) ? 64 : (C % 32 == 0 ? 32 : 0);
    return C % 32 == 0 ? 32 : (C % 16 == 0 ? 16 : 0);
}

// Chooses the tile rectangle Wt x R (Wt * R <= 128) that fills most of the 128 tile rows with pixels of
// the grid.  Every box starts a multiple of Wt rows into the stage and the copy engine wants 128-byte
// alignment there, so Wt * row_bytes_min must be a multiple of 128.
bool make_grid(RowGrid &g, int Wr, int Hr, int Nimg, int row_bytes_min) {
    g.Wr = Wr; g.Hr = Hr; g.Nimg = Nimg;
    const long long rows = (long long)Nimg * Hr;
    const int wstep = row_bytes_min >= 128 ? 1 : 128 / row_bytes_min;
    long long best = -1;
    for (int xs = (Wr + 127) / 128; xs <= (Wr + 127) / 128 + 7 && xs <= Wr; ++xs) {
        int Wt = (Wr + xs - 1) / xs;
        Wt = (Wt + wstep - 1) / wstep * wstep;
        if (Wt > 128) continue;
        int R = 128 / Wt;
        if (R > kMaxBoxes) R = kMaxBoxes;
        if (R > rows) R = (int)rows;
        const int xsegs = (Wr + Wt - 1) / Wt;
        const long long util = (long long)Wr * R * 1000 / ((long long)xsegs * 128);  // useful share of tile rows
        // narrower tiles mean more and smaller boxes: only worth a clear gain, and never below 16 pixels
        if (best < 0 || (Wt >= 16 && util * 10 > best * 11)) {
            best = util;
            g.Wt = Wt; g.xsegs = xsegs; g.R = R;
        }
    }
    if (best < 0) return false;
    const long long tiles = (rows + g.R - 1) / g.R * g.xsegs;
    if (tiles > 0x3fffffff) return false;
    g.tiles = (int)tiles;
    g.arows = g.R * g.Wt;
    return true;
}

// Maps of an activation tensor [Nimg][Hs][Ws][C, row stride ld] for boxes of CB channels, the tile width of
// `g` and heights 1 .. min(R, Hr) rows, traversal stride es along W and H.
int make_act_maps(CUtensorMap *maps, const bf16 *base, int C, long long ld, int Ws, int Hs, int Nimg,
                  const RowGrid &g, int CB, int es) {
    const long long dims[4] = {C, Ws, Hs, Nimg};
    const int wbox = g.Wt * es;
    const int maxh = g.R < g.Hr ? g.R : g.Hr;
    for (int i = 0; i < maxh; ++i) {
        const int box[4] = {CB, wbox, (i + 1) * es, 1};
        const int estr[4] = {1, es, es, 1};
        const int s = make_map(&maps[i], base, 4, dims, ld, box, estr, CB * 2);
        if (s != PPO_OK) return s;
    }
    return PPO_OK;
}

int stages_for(size_t stage_bytes) {
    int s = (int)(kSmemBudget / stage_bytes);
    return s > kMaxStages ? kMaxStages : s;
}

int pick_bn(int N) {  // tile width: N split evenly into tiles of at most 256, rounded up to 16
    const int tiles = (N + 255) / 256;
    int bn = ((N + tiles - 1) / tiles + 15) / 16 * 16;
    return bn < 16 ? 16 : bn;
}

// Tile width of a flat GEMM (rows x N): as pick_bn, then halved while the tiles would leave more than half of the SMs
// without work (few rows, as in the per-step products of a recurrent layer) and the halves still divide N.
static int flat_bn(int N, long long rows) {
    int bn = pick_bn(N);
    const long long mt = (rows + 127) / 128;
    while (bn >= 64 && bn % 32 == 0 && N % (bn / 2) == 0 && mt * ((N + bn - 1) / bn) < ppo_num_sms() / 2) bn /= 2;
    return bn;
}

int ensure_smem_attrs() {
    static bool attr_set[64] = {false};
    int dev = 0;
    PPO_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return PPO_ERR_CUDA;
    if (!attr_set[dev]) {
        const int mx = (int)(kSmemBudget + sizeof(PipeK) + 1024);
        PPO_CUDA_CHECK(cudaFuncSetAttribute(tma_kmajor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax));
        PPO_CUDA_CHECK(cudaFuncSetAttribute(tma_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, mx));
        attr_set[dev] = true;
    }
    return PPO_OK;
}

// Most A boxes any tile of the grid is cut into (the cut repeats with the tile's first row modulo Hr).
int max_boxes(const RowGrid &g) {
    Box tmp[kMaxBoxes];
    int mx = 1;
    const int groups = g.tiles / g.xsegs;  // the cut depends on the row group only
    const int lim = groups < g.Hr + 1 ? groups : g.Hr + 1;
    for (int t = 0; t < lim; ++t) {
        const int n = build_boxes(g, t * g.xsegs, tmp);
        mx = n > mx ? n : mx;
    }
    const int n = build_boxes(g, g.tiles - 1, tmp);
    return n > mx ? n : mx;
}

// `a.wtaps` = taps of the whole weight tensor (all classes).
int launch_kmajor(KArgs &a, cudaStream_t st) {
    int s = ensure_smem_attrs();
    if (s != PPO_OK) return s;
    a.tiles_n = (a.N + a.BN - 1) / a.BN;
    if (a.mode != EPI_DGRAD && a.tiles_n * a.BN > kMaxBias) return PPO_ERR_UNSUPPORTED;  // bias staged in shared memory
    const long long per = (long long)a.grid.tiles * a.tiles_n;
    const long long total = per * a.ncls;
    if (total <= 0) return PPO_OK;
    if (total > 0x7fffffffll) return PPO_ERR_UNSUPPORTED;
    a.total_tiles = (int)total;
    a.nbmax = max_boxes(a.grid);
    const size_t b_bytes = (size_t)a.BN * a.row_bytes;
    const size_t res = (size_t)a.wtaps * a.kchunks * b_bytes;
    // resident weights only while they leave most of the shared memory to the A stages: the bytes in flight
    // are what hides the copy latency
    a.wres = (a.tiles_n == 1 && a.ncls == 1 && res <= kMaxResident && a.wtaps * a.kchunks <= kMaxWtab) ? 1 : 0;
    // Narrow tiles (BN <= 128) leave the tensor pipe mostly idle because one thread per CTA cannot issue MMAs
    // fast enough; two CTAs per SM (half the shared and tensor memory each, 8 epilogue warps each) double the
    // issue rate.  Wide tiles run at the tensor rate with one CTA and keep the SM to themselves.
    // A GEMM of a few row tiles gives a CTA one or two tiles: nothing amortises the copy latency, so such a CTA takes the
    // SM alone, with stages of up to 96 KB (fewer, larger hand-overs), and the narrow-tile rule below does not apply.
    const bool small_m = a.grid.tiles <= 4 && (a.ncls == 1 || a.cls_orows != 0);
    const bool two = a.BN <= 128 && !small_m;
    a.tmem_cap = two ? 256 : 512;
    a.nepi = (!two && a.mode == EPI_DGRAD && a.mask_bits) ? 16 : 8;
    const size_t fixed = sizeof(PipeK) + (size_t)a.nepi * 2048 + 1024;  // pipeline state, epilogue staging, alignment slack
    const size_t cta_max = two ? kSmemMax / 2 : kSmemMax;
    if (a.wres && res + fixed + 3 * (size_t)128 * a.row_bytes + 1024 > cta_max) a.wres = 0;
    const size_t sub = (size_t)128 * a.row_bytes + (a.wres ? 0 : b_bytes);
    const size_t budget = cta_max - 1024 - fixed - (a.wres ? res : 0);
    int G = (int)(((small_m ? 96 : 48) * 1024) / sub);  // sub-blocks per stage: fewer barrier round trips per byte
    G = G < 1 ? 1 : (G > 8 ? 8 : G);
    while (G > 1 && budget / (G * sub) < (small_m ? 2 : 3)) --G;
    const int lps = a.nbmax + (a.wres ? 0 : 1);  // copies per sub-block; one producer lane each
    if (lps > 32) return PPO_ERR_UNSUPPORTED;
    while (G > 1 && G * lps > 32) --G;
    a.G = G;
    a.stages = (int)(budget / (G * sub));
    if (a.stages > kMaxStages) a.stages = kMaxStages;
    if (a.stages < 2) return PPO_ERR_UNSUPPORTED;
    const int sms = ppo_num_sms();
    const long long ctas = two ? 2ll * sms : sms;
    const unsigned grid = (unsigned)(total < ctas ? total : ctas);
    const size_t smem = (size_t)a.stages * G * sub + (a.wres ? res : 0) + fixed;
    tma_kmajor_kernel<<<grid, (2 + a.nepi) * 32, smem, st>>>(a);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

bool is_flat(const ConvGeom &g) { return g.Hi == 1 && g.Wi == 1 && g.Ho == 1 && g.Wo == 1 && g.k == 1; }

}  // namespace

int tma_gemm_fwd(const ConvGeom &g, const bf16 *X, const bf16 *W, const FwdEpilogue &e, int32_t *status,
                 cudaStream_t st) {
    if (!status || g.taps() > kMaxTaps || g.Ci % 8 != 0) return PPO_ERR_UNSUPPORTED;
    const bool flat = is_flat(g);
    const int CB = channels_per_box(g.Ci, flat);
    if (CB == 0) return PPO_ERR_UNSUPPORTED;
    KArgs a = {};
    a.CB = CB;
    a.row_bytes = CB * 2;
    a.kchunks = (g.Ci + CB - 1) / CB;
    a.w_tap = g.Ci;
    a.wtaps = g.taps();
    // a fully connected layer is one image with a single row of B pixels
    const bool ok = flat ? make_grid(a.grid, g.B, 1, 1, a.row_bytes) : make_grid(a.grid, g.Wo, g.Ho, g.B, a.row_bytes);
    if (!ok) return PPO_ERR_UNSUPPORTED;
    int s = flat ? make_act_maps(a.mapA, X, g.Ci, g.Ci, g.B, 1, 1, a.grid, CB, 1)
                 : make_act_maps(a.mapA, X, g.Ci, g.Ci, g.Wi, g.Hi, g.B, a.grid, CB, 2);
    if (s != PPO_OK) return s;
    a.N = g.Co;
    a.BN = flat && e.out ? flat_bn(g.Co, g.B) : pick_bn(g.Co);
    {
        const long long dims[2] = {g.K(), g.Co};
        const int box[2] = {CB, a.BN}, es[2] = {1, 1};
        s = make_map(&a.mapB, W, 2, dims, g.K(), box, es, a.row_bytes);
        if (s != PPO_OK) return s;
    }
    a.s_mul = flat ? 1 : 2;
    a.s_oy = a.s_ox = -g.pad;
    a.Hout = flat ? 1 : g.Ho;
    a.Wout = flat ? g.B : g.Wo;
    a.ldo = e.ldo ? e.ldo : g.Co;
    a.mode = e.out ? EPI_FWD : EPI_HEAD;
    if (e.ln_gamma) {
        if (!e.ln_beta || !e.ln_xhat || !e.ln_rstd || !e.out || g.Co > 256 || g.Co % 32 != 0 || a.ldo != g.Co) return PPO_ERR_UNSUPPORTED;
        a.ln_gamma = e.ln_gamma;
        a.ln_beta = e.ln_beta;
        a.ln_xhat = e.ln_xhat;
        a.ln_rstd = e.ln_rstd;
    }
    a.relu = e.relu;
    a.A = e.A;
    a.bias = e.bias;
    a.out = e.out;
    a.mean = e.out_mean;
    a.out_bits = (e.out_bits && e.relu && g.Co % 32 == 0) ? e.out_bits : nullptr;
    if (e.out_bits && !a.out_bits) return PPO_ERR_UNSUPPORTED;
    a.value = e.out_value;
    a.status = status;
    if (a.mode == EPI_FWD && g.Co % 8 != 0) return PPO_ERR_UNSUPPORTED;
    a.ncls = 1;
    KClass &k = a.cls[0];
    k.b_row0 = 0;
    k.taps.n = g.taps();
    for (int t = 0; t < g.taps(); ++t) {
        k.taps.dy[t] = (signed char)(t / g.k);
        k.taps.dx[t] = (signed char)(t % g.k);
        k.taps.wt[t] = (short)t;
    }
    return launch_kmajor(a, st);
}

static void tma_dgrad_shifts(int k, int *dmin, int *n1) {
    const int pad = k / 2;
    *dmin = -((k - 1 - pad) / 2);
    *n1 = (1 + pad) / 2 - *dmin + 1;
}

// Fully connected layers: dX[b][ci] = sum_co dY[b][co] Wt[ci][co].  Convolutions: the four stride-parity
// classes of input pixels are computed together.  Row (y, x) of the GEMM stands for the 2x2 block of input
// pixels (2y + ph, 2x + pw); column class * Ci + ci; the reduction runs over the shifts (dy, dx) of the
// output pixel (y + dy, x + dx) and its channels, with the weights Wc[class * Ci + ci][shift][co] (zero
// where a class has no kernel tap at that shift).  One wide GEMM instead of four narrow ones: the tensor
// core is fed by one thread, and an instruction of 64 columns or fewer occupies it as long as one of 128
// (~55 cycles per issue at best; 128 columns run at the tensor rate of 64 cycles, 256 at 128).
int tma_gemm_dgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *Wt, int wt_ld, const bf16 *Wc,
                   const DgradEpilogue &e, int32_t *status, cudaStream_t st) {
    if (!status || g.Ci % 8 != 0 || ldy % 8 != 0 || wt_ld % 8 != 0 || ldy < wt_ld) return PPO_ERR_UNSUPPORTED;
    const bool flat = is_flat(g);
    // a 32-column group of the staged epilogue must lie inside one parity class; with 16 input channels the
    // per-thread epilogue (16 columns = one class at a time) takes over, which needs the bf16 gate
    if (!flat && (g.k < 3 || g.Hi < 2 || g.Wi < 2 || !Wc)) return PPO_ERR_UNSUPPORTED;
    if (!flat && g.Ci % 32 != 0 && (g.Ci % 16 != 0 || !e.mask_act || e.mask_bits || !e.out)) return PPO_ERR_UNSUPPORTED;
    const int CB = channels_per_box(g.Co, flat);
    if (CB == 0 || g.taps() > kMaxTaps || wt_ld < g.Co) return PPO_ERR_UNSUPPORTED;
    KArgs a = {};
    a.CB = CB;
    a.row_bytes = CB * 2;
    a.kchunks = (g.Co + CB - 1) / CB;
    a.w_tap = wt_ld;
    const int Hr = flat ? 1 : (g.Hi + 1) / 2, Wr = flat ? g.B : (g.Wi + 1) / 2;
    if (!make_grid(a.grid, Wr, Hr, flat ? 1 : g.B, a.row_bytes)) return PPO_ERR_UNSUPPORTED;
    int s = flat ? make_act_maps(a.mapA, dY, g.Co, ldy, g.B, 1, 1, a.grid, CB, 1)
                 : make_act_maps(a.mapA, dY, g.Co, ldy, g.Wo, g.Ho, g.B, a.grid, CB, 1);
    if (s != PPO_OK) return s;
    a.s_mul = 1;
    a.s_oy = a.s_ox = 0;
    a.Hout = flat ? 1 : g.Hi;
    a.Wout = flat ? g.B : g.Wi;
    a.ldo = g.Ci;
    a.mode = EPI_DGRAD;
    a.out = e.out;
    a.out_f32 = e.out_f32;
    a.mask = e.mask_act;
    a.mask_bits = flat ? nullptr : e.mask_bits;
    a.status = status;
    const int ks = flat && e.ksplit > 1 ? e.ksplit : 1;
    if (ks > 1) {
        // Split reduction: the Co columns of dY are seen as an image of ks rows of Co / ks channels (row y of pixel x
        // starts at x * ldy + y * Co / ks), class s reads row s against the weight columns s * Co / ks .. and
        // leaves its product in its own copy of the output.
        if (ks > 4 || g.Co % (ks * 64) != 0 || !e.out_f32 || e.out || e.mask_act) return PPO_ERR_UNSUPPORTED;
        const int Kc = g.Co / ks;
        a.kchunks = Kc / CB;
        a.w_tap = Kc;
        EncodeTiledFn fn = encode_fn();
        if (!fn || !ppo_aligned(dY, 16)) return PPO_ERR_UNSUPPORTED;
        const cuuint64_t gd[4] = {(cuuint64_t)Kc, (cuuint64_t)g.B, (cuuint64_t)ks, 1};
        const cuuint64_t gs[3] = {(cuuint64_t)ldy * 2, (cuuint64_t)Kc * 2, (cuuint64_t)ldy * 2 * (cuuint64_t)g.B};
        const cuuint32_t bx[4] = {(cuuint32_t)CB, (cuuint32_t)a.grid.Wt, 1, 1}, es[4] = {1, 1, 1, 1};
        if (a.grid.R != 1 ||
            fn(&a.mapA[0], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<bf16 *>(dY), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PPO_ERR_UNSUPPORTED;
        a.N = g.Ci;
        a.BN = flat_bn(g.Ci, (long long)g.B * ks);
        a.wtaps = ks;
        const long long dims[2] = {wt_ld, g.Ci};
        const int box[2] = {CB, a.BN}, esb[2] = {1, 1};
        s = make_map(&a.mapB, Wt, 2, dims, wt_ld, box, esb, a.row_bytes);
        if (s != PPO_OK) return s;
        a.ncls = ks;
        a.cls_orows = g.B;
        for (int c = 0; c < ks; ++c) {
            KClass &k = a.cls[c];
            k.b_row0 = 0;
            k.taps.n = 1;
            k.taps.dy[0] = (int8_t)c;
            k.taps.dx[0] = 0;
            k.taps.wt[0] = (decltype(k.taps.wt[0]))c;
        }
        return launch_kmajor(a, st);
    }
    if (flat) {
        a.N = g.Ci;
        a.BN = flat_bn(g.Ci, g.B);
        a.wtaps = 1;
        const long long dims[2] = {wt_ld, g.Ci};
        const int box[2] = {CB, a.BN}, es[2] = {1, 1};
        s = make_map(&a.mapB, Wt, 2, dims, wt_ld, box, es, a.row_bytes);
        if (s != PPO_OK) return s;
        a.ncls = 1;
        KClass &k = a.cls[0];
        k.b_row0 = 0;
        k.taps.n = 1;
        k.taps.dy[0] = k.taps.dx[0] = 0;
        k.taps.wt[0] = 0;
        return launch_kmajor(a, st);
    }
    int dmin, n1;
    tma_dgrad_shifts(g.k, &dmin, &n1);
    const int nshift = n1 * n1, Ntot = 4 * g.Ci;
    // 256 or 512 merged columns (C_in = 64, 128) go as groups of 128: a group takes only the shifts at which its
    // parity classes have taps (6 of 8 group-shift pairs for two groups, 9 of 16 for four: one per kernel tap),
    // so the multiplications by zero weights of a single wide GEMM fall away, at the same operand bytes, and tiles
    // of 128 columns run two CTAs per SM
    a.BN = (Ntot == 256 || Ntot == 512) ? 128 : pick_bn(Ntot);
    if (Ntot % a.BN != 0 || Ntot / a.BN > 4 || nshift > kMaxTaps) return PPO_ERR_UNSUPPORTED;
    a.N = a.BN;  // every group is one full tile of columns
    a.nq_ci = g.Ci;
    a.wtaps = nshift;
    {
        const long long dims[2] = {(long long)nshift * wt_ld, Ntot};
        const int box[2] = {CB, a.BN}, es[2] = {1, 1};
        s = make_map(&a.mapB, Wc, 2, dims, (long long)nshift * wt_ld, box, es, a.row_bytes);
        if (s != PPO_OK) return s;
    }
    a.ncls = Ntot / a.BN;
    for (int c = 0; c < a.ncls; ++c) {
        KClass &k = a.cls[c];
        k.b_row0 = c * a.BN;
        const int q_lo = c * a.BN / g.Ci, q_hi = ((c + 1) * a.BN - 1) / g.Ci;
        int nt = 0;
        for (int sy = 0; sy < n1; ++sy)
            for (int sx = 0; sx < n1; ++sx) {
                bool used = false;
                for (int q = q_lo; q <= q_hi; ++q) {
                    const int kh = (q >> 1) + g.pad - 2 * (dmin + sy), kw = (q & 1) + g.pad - 2 * (dmin + sx);
                    used = used || (kh >= 0 && kh < g.k && kw >= 0 && kw < g.k);
                }
                if (!used) continue;
                k.taps.dy[nt] = (signed char)(dmin + sy);
                k.taps.dx[nt] = (signed char)(dmin + sx);
                k.taps.wt[nt] = (short)(sy * n1 + sx);
                ++nt;
            }
        if (nt == 0) return PPO_ERR_UNSUPPORTED;
        k.taps.n = nt;
    }
    return launch_kmajor(a, st);
}

size_t tma_dgrad_weight_elems(int Ci, int k, int wt_ld) {
    int dmin, n1;
    tma_dgrad_shifts(k, &dmin, &n1);
    return (size_t)4 * Ci * n1 * n1 * wt_ld;
}

// Wc[class * Ci + ci][shift][co (row stride ld)] = W[co][kh][kw][ci] with kh = ph + pad - 2 dy, kw = pw + pad - 2 dx
// when that tap exists, else 0.
__global__ void __launch_bounds__(256) dgrad_weights_kernel(const bf16 *__restrict__ W, bf16 *__restrict__ Wc, int Co,
                                                            int k, int Ci, int ld, int dmin, int n1) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)4 * Ci * n1 * n1 * ld;
    if (i >= total) return;
    const int co = (int)(i % ld);
    long long r = i / ld;
    const int sh = (int)(r % (n1 * n1));
    r /= n1 * n1;
    const int ci = (int)(r % Ci), q = (int)(r / Ci);
    const int pad = k / 2;
    const int kh = (q >> 1) + pad - 2 * (dmin + sh / n1), kw = (q & 1) + pad - 2 * (dmin + sh % n1);
    const bool v = co < Co && kh >= 0 && kh < k && kw >= 0 && kw < k;
    Wc[i] = v ? W[(((size_t)co * k + kh) * k + kw) * Ci + ci] : __float2bfloat16_rn(0.f);
}

int tma_dgrad_weights(const bf16 *W, bf16 *Wc, int Co, int k, int Ci, int wt_ld, cudaStream_t st) {
    int dmin, n1;
    tma_dgrad_shifts(k, &dmin, &n1);
    const long long total = (long long)tma_dgrad_weight_elems(Ci, k, wt_ld);
    dgrad_weights_kernel<<<ppo_cdiv(total, 256), 256, 0, st>>>(W, Wc, Co, k, Ci, wt_ld, dmin, n1);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

int wgrad_reduce(const float *part, int jtiles, int ctiles, int splits, int BN, int Kfwd, int Co, float *dW, float *db,
                 int ones_row, cudaStream_t st) {
    const long long n = (long long)Co * Kfwd + (db ? Co : 0);
    wgrad_reduce_kernel<<<ppo_cdiv(n, 256), 256, 0, st>>>(part, jtiles, ctiles, splits, BN, Kfwd, Co, dW, db, ones_row);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}

int tma_gemm_wgrad(const ConvGeom &g, const bf16 *dY, int ldy, const bf16 *X, float *dW, float *db, float *part,
                   size_t part_elems, int32_t *status, cudaStream_t st) {
    if (!status || !part || g.Ci % 8 != 0 || ldy % 8 != 0 || g.taps() > kMaxTaps) return PPO_ERR_UNSUPPORTED;
    const bool flat = is_flat(g);
    const int CB = channels_per_box(g.Ci, flat);
    const int CBn = g.Co % 64 == 0 ? 64 : (g.Co % 32 == 0 ? 32 : 0);
    if (CB == 0 || CBn == 0) return PPO_ERR_UNSUPPORTED;
    WArgs a = {};
    a.CB = CB;
    a.rbA = CB * 2;
    a.mblocks = 128 / CB;
    a.kchunks = (g.Ci + CB - 1) / CB;
    a.CBn = CBn;
    a.rbB = CBn * 2;
    a.BN = g.Co < 256 ? g.Co : 256;
    if (g.Co % a.BN != 0 || a.BN % CBn != 0) return PPO_ERR_UNSUPPORTED;
    a.nblocks = a.BN / CBn;
    const int rb_min = a.rbA < a.rbB ? a.rbA : a.rbB;
    const bool ok = flat ? make_grid(a.grid, g.B, 1, 1, rb_min) : make_grid(a.grid, g.Wo, g.Ho, g.B, rb_min);
    if (!ok) return PPO_ERR_UNSUPPORTED;
    int s = flat ? make_act_maps(a.mapA, X, g.Ci, g.Ci, g.B, 1, 1, a.grid, CB, 1)
                 : make_act_maps(a.mapA, X, g.Ci, g.Ci, g.Wi, g.Hi, g.B, a.grid, CB, 2);
    if (s != PPO_OK) return s;
    s = flat ? make_act_maps(a.mapB, dY, g.Co, ldy, g.B, 1, 1, a.grid, CBn, 1)
             : make_act_maps(a.mapB, dY, g.Co, ldy, g.Wo, g.Ho, g.B, a.grid, CBn, 1);
    if (s != PPO_OK) return s;
    a.s_mul = flat ? 1 : 2;
    a.pad = g.pad;
    a.ksz = g.k;
    a.ntaps = g.taps();
    a.Kfwd = g.K();
    a.Co = g.Co;
    a.nmma = (a.grid.arows + 15) / 16;
    a.part = part;
    a.status = status;
    const size_t stage = (size_t)128 * 256 + (size_t)128 * 2 * a.BN;
    // two CTAs per SM (twice the MMA issue rate) when two stages fit into half of the shared memory
    const size_t half_budget = kSmemMax / 2 - 1024 - sizeof(Pipe) - 1024;
    const bool two = 2 * stage <= half_budget && a.BN <= 256;
    a.stages = two ? (int)(half_budget / stage) : stages_for(stage);
    if (a.stages > kMaxStages) a.stages = kMaxStages;
    if (a.stages < 2) return PPO_ERR_UNSUPPORTED;
    s = ensure_smem_attrs();
    if (s != PPO_OK) return s;
    int jtiles = (a.ntaps * a.kchunks + a.mblocks - 1) / a.mblocks;
    const int ctiles = g.Co / a.BN;
    if (db) {
        // the ones column goes into the first unused block of the last column tile; when every block is
        // taken, one more tile carries it alone
        if (flat || g.Ci % CB != 0) return PPO_ERR_UNSUPPORTED;
        a.has_db = 1;
        a.ones_blk = a.ntaps * a.kchunks - (jtiles - 1) * a.mblocks;
        if (a.ones_blk == a.mblocks) {
            a.ones_blk = 0;
            ++jtiles;
        }
    }
    int splits = (two ? 2 : 1) * ppo_num_sms() / (jtiles * ctiles);
    if (splits < 1) splits = 1;
    const size_t per_split = (size_t)jtiles * ctiles * 128 * a.BN;
    if ((size_t)splits * per_split > part_elems) splits = (int)(part_elems / per_split);  // the scratch bounds the split
    if (splits < 1) return PPO_ERR_SHAPE;
    if (splits > a.grid.tiles) splits = a.grid.tiles;
    a.tiles_per_split = (a.grid.tiles + splits - 1) / splits;
    splits = (a.grid.tiles + a.tiles_per_split - 1) / a.tiles_per_split;  // every split has at least one pixel tile
    dim3 grid((unsigned)jtiles, (unsigned)ctiles, (unsigned)splits);
    tma_wgrad_kernel<<<grid, kThreads, (size_t)a.stages * stage + sizeof(Pipe) + 1024, st>>>(a);
    PPO_LAUNCH_CHECK();
    return wgrad_reduce(part, jtiles, ctiles, splits, a.BN, a.Kfwd, g.Co, dW, db,
                        db ? (jtiles - 1) * 128 + a.ones_blk * CB : 0, st);
}

// Scratch floats that let a weight-gradient GEMM of this shape split as far as it wants: every CTA of a grid of up
// to two per SM (or one per tile, if that is more) leaves a 128 x BN tile.
size_t wgrad_scratch_elems(const ConvGeom &g) {
    const int BN = g.Co < 256 ? (g.Co + 15) / 16 * 16 : 256;
    const long long tiles = (long long)((g.K() + 127) / 128 + 1) * ((g.Co + BN - 1) / BN);
    const long long ctas = tiles > 2ll * ppo_num_sms() ? tiles : 2ll * ppo_num_sms();
    return (size_t)ctas * 128 * BN;
}
