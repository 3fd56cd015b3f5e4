// Tensor-core convolution for sm_100a: implicit GEMM with bf16 operands, fp32 accumulation in
// tensor memory (tcgen05.mma), operand tiles staged in shared memory by TMA.
//
//   out[p, co] = sum_{tap, ci} a[p (+) tap, ci] * Wp[co, tap, ci]        (Eq. 2, Conv_kxk; stride 1)
//
// GEMM view: M = 128 output pixels per CTA (whole image rows, so a tile is one TMA box of the NHWC
// tensor), N = output channels, K = taps x input channels.  For every tap the A tile is the same
// box shifted by (kh - pad, kw - pad); TMA zero-fills what falls outside the image, which is
// exactly the convolution's zero padding because the activated tensor is materialised.
// dgrad is the same kernel run on the upstream gradient with the tap-mirrored, transposed pack
// of the weights.  Each entry point returns false for shapes it does not take.
//
// Roles inside a CTA (192 threads): warp 0 issues TMA loads, warp 1 allocates tensor memory and
// issues the MMAs, warps 2..5 drain the accumulator (tcgen05.ld), apply the coupling epilogue
// (out = partner +/- acc on the float or fixed-point state) and store.
// Every mbarrier wait is bounded; on expiry the kernel records a status word and leaves.
#include "common.cuh"
#include "tc_ptx.cuh"
#include "conv_epilogue.cuh"
#include <cuda.h>
#include <string.h>

using namespace tc;

namespace {

constexpr int kStages = 4;
constexpr int kThreads = 192;

struct TcParams {
    int taps;        // k*k
    int k;           // kernel size
    int chunks;      // channel chunks per tap
    int KC;          // channels per chunk (16, 32 or 64)
    int cin_pad;     // chunks * KC
    int BN;          // N tile
    int stride;      // 1 or 2: input pixel = output pixel * stride + tap - pad (TMA traversal stride)
    TileGeom g;      // output tiles
    EpiArgs epi;
    int *status;
};

struct __align__(8) TcShared {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t failed;
    RowMap rows;
};

// Persistent CTA: walks the pixel tiles blockIdx.x, blockIdx.x + gridDim.x, ... of N tile blockIdx.y.
// The operand ring runs on across tiles; the accumulator alternates between two tensor-memory
// buffers so that the epilogue of one tile overlaps the MMAs of the next.
__global__ void __launch_bounds__(kThreads, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // operand stages first (1024-byte aligned for the 128-byte swizzle), epilogue stage and bookkeeping behind them
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int box_px = p.g.BIMG * p.g.BH * p.g.W;
    const int a_bytes = box_px * p.KC * 2, b_bytes = p.BN * p.KC * 2;
    const int b_off = (128 * p.KC * 2 + 1023) & ~1023;
    const int stage_bytes = b_off + ((b_bytes + 1023) & ~1023);
    float *estage = (float *)(tiles + kStages * stage_bytes);
    TcShared *sh = (TcShared *)((uint8_t *)estage + kEpiStageBytes + kEpiSumFloats * 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int iters = p.taps * p.chunks;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * p.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; s++) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&sh->acc_full[b], 1); mbar_init(&sh->acc_empty[b], 128); }
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_a); tma_prefetch_desc(&map_b);
    }
    if (warp == 1) tmem_alloc(&sh->tmem_base, tmem_cols);
    if (warp >= 2) build_row_map(p.g, &sh->rows, ((warp & 3) << 5) | lane);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_enter();             // the set-up above may overlap the kernel before; its outputs are read from here on
    const uint32_t tmem_d = sh->tmem_base;
    const int col0 = blockIdx.y * p.BN;
    const int pad = p.k / 2;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t itg = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < p.g.n_px_tiles && ok; t += gridDim.x) {
                int n0, h0;
                tile_origin(p.g, t, n0, h0);
                for (int it = 0; it < iters; it++, itg++) {
                    const int s = itg % kStages; const uint32_t round = itg / kStages;
                    if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                    const int tap = it / p.chunks, ch = it - tap * p.chunks;
                    const int kh = tap / p.k, kw = tap - kh * p.k;
                    uint8_t *sa = tiles + s * stage_bytes;
                    mbar_expect_tx(&sh->full[s], (uint32_t)(a_bytes + b_bytes));
                    tma_load_4d(sa, &map_a, &sh->full[s], ch * p.KC, kw - pad, h0 * p.stride + kh - pad, n0);
                    tma_load_2d(sa + b_off, &map_b, &sh->full[s], tap * p.cin_pad + ch * p.KC, col0);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(p.BN);
            const int row_bytes = p.KC * 2;
            uint32_t itg = 0;
            bool ok = true;
            int ti = 0;
            for (int t = blockIdx.x; t < p.g.n_px_tiles && ok; t += gridDim.x, ti++) {
                const int buf = ti & 1; const uint32_t use = ti >> 1;
                if (use > 0 && !mbar_wait(&sh->acc_empty[buf], (use - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                tc_fence_after();
                const uint32_t acc = tmem_d + (uint32_t)(buf * p.BN);
                for (int it = 0; it < iters; it++, itg++) {
                    const int s = itg % kStages; const uint32_t round = itg / kStages;
                    if (!mbar_wait(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(tiles + s * stage_bytes);
                    for (int kk = 0; kk < p.KC / 16; kk++) {
                        const uint64_t da = smem_desc(sa + kk * 32, row_bytes);
                        const uint64_t db = smem_desc(sa + b_off + kk * 32, row_bytes);
                        mma_bf16(acc, da, db, idesc, (it > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(&sh->empty[s]);          // frees the stage once these MMAs have read it
                }
                if (ok) mma_commit(&sh->acc_full[buf]);
            }
        }
    } else {
        // epilogue: this warp may touch accumulator lanes 32*(warp%4) .. +31
        const int etid = ((warp & 3) << 5) | lane;
        float *esums = estage + 128 * kEpiPitch;
        epilogue_init(esums, etid);
        named_barrier(1, 128);
        bool ok = true;
        int ti = 0;
        for (int t = blockIdx.x; t < p.g.n_px_tiles; t += gridDim.x, ti++) {
            const int buf = ti & 1; const uint32_t use = ti >> 1;
            int n0, h0;
            tile_origin(p.g, t, n0, h0);
            EpiPrefetch pre;
            epilogue_prefetch(p.epi, p.BN, col0, &sh->rows, p.g, n0, h0, etid, pre);     // before the accumulator is ready
            if (etid == 0) ok = mbar_wait(&sh->acc_full[buf], use & 1) && sh->failed == 0;     // one thread polls, the rest block
            ok = named_barrier_and(2, 128, ok);
            if (!ok) break;
            tc_fence_after();
            epilogue_tile(p.epi, tmem_d + (uint32_t)(buf * p.BN), p.BN, col0, &sh->rows, p.g, n0, h0, estage, esums, etid, &sh->acc_empty[buf], pre);
        }
        if (ok) epilogue_finish(p.epi, p.BN, col0, estage, esums, etid);
        else if (lane == 0) atomicExch(&sh->failed, 1u);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && sh->failed) atomicExch(p.status, (int)REVNET_E_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, tmem_cols);
    }
}

// ---- weight packs: bf16 [rows_pad][taps][cin_pad]; transposed = true builds the dgrad operand
// (rows = input channels, columns = output channels, taps mirrored)
__global__ void pack_weights_kernel(const float *__restrict__ W, bf16 *__restrict__ out, int Co, int Ci, int k,
                                    int rows_pad, int cols_pad, int transposed) {
    pdl_enter();
    const int taps = k * k;
    const size_t n = (size_t)rows_pad * taps * cols_pad;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % cols_pad);
        const int tap = (int)((i / cols_pad) % taps);
        const int r = (int)(i / ((size_t)cols_pad * taps));
        float v = 0.f;
        if (!transposed) { if (r < Co && c < Ci) v = W[((size_t)r * taps + tap) * Ci + c]; }
        else { if (r < Ci && c < Co) v = W[((size_t)c * taps + (taps - 1 - tap)) * Ci + r]; }
        out[i] = __float2bfloat16_rn(v);
    }
}

// all packs of a step in one launch: blockIdx.y walks the job table
__global__ void pack_weights_batch_kernel(const PackJob *__restrict__ jobs) {
    pdl_enter();
    const PackJob j = jobs[blockIdx.y];
    const int taps = j.k * j.k;
    const size_t n = (size_t)j.rows_pad * taps * j.cols_pad;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % j.cols_pad);
        const int tap = (int)((i / j.cols_pad) % taps);
        const int r = (int)(i / ((size_t)j.cols_pad * taps));
        float v = 0.f;
        if (!j.transposed) { if (r < j.Co && c < j.Ci) v = j.W[((size_t)r * taps + tap) * j.Ci + c]; }
        else { if (r < j.Ci && c < j.Co) v = j.W[((size_t)c * taps + (taps - 1 - tap)) * j.Ci + r]; }
        j.out[i] = __float2bfloat16_rn(v);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encoder(revnet_ctx *ctx) {
    if (!ctx->encode_tiled) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || qres != cudaDriverEntryPointSuccess)
            fn = nullptr;
        ctx->encode_tiled = fn;
    }
    return (EncodeTiledFn)ctx->encode_tiled;
}

int round_up(int x, int m) { return (x + m - 1) / m * m; }

// 128-row tiles over an output of N x H x W pixels: whole rows of one image (the last tile of an
// image may be ragged), or whole images when an image has at most 64 pixels.  Rows of the tile
// that fall outside are padding: TMA fills their operand rows with zeros and the epilogue skips them.
bool tile_geom(Geom g, TileGeom &t) {
    if (g.W > 128 || g.W < 1) return false;
    t.N = g.N; t.H = g.H; t.W = g.W; t.hw_order = 0; t.Wp = g.W;
    t.BH = 128 / g.W; if (t.BH > g.H) t.BH = g.H;
    t.BIMG = 1;
    if (t.BH == g.H) { t.BIMG = 128 / (g.H * g.W); if (t.BIMG > g.N) t.BIMG = g.N; if (t.BIMG < 1) t.BIMG = 1; }
    t.tiles_per_img = (g.H + t.BH - 1) / t.BH;
    t.n_px_tiles = t.BIMG > 1 ? (g.N + t.BIMG - 1) / t.BIMG : g.N * t.tiles_per_img;
    return true;
}

struct TcShape { int KC, cin_pad, chunks, BN, n_tiles, smem; TileGeom g; };

// Which shapes the kernel takes: stride 1 or 2, k in {1,3}, channel rows 16-byte aligned for TMA.
bool tc_shape(Geom g, int cin, int cout, int k, int stride, TcShape &s) {   // g: output geometry
    if ((stride != 1 && stride != 2) || (k != 1 && k != 3) || cin % 8 || cout % 4) return false;
    if (!tile_geom(g, s.g)) return false;
    if (s.g.W * stride > 256 || s.g.BH * stride > 256) return false;
    s.cin_pad = round_up(cin, 16);
    s.KC = s.cin_pad % 64 == 0 ? 64 : (s.cin_pad % 32 == 0 ? 32 : 16);
    s.chunks = s.cin_pad / s.KC;
    const int cout_pad = round_up(cout, 16);
    s.BN = cout_pad <= 128 ? cout_pad : 128;
    s.n_tiles = (cout_pad + s.BN - 1) / s.BN;
    const int a_bytes = 128 * s.KC * 2, b_bytes = s.BN * s.KC * 2;
    s.smem = 1024 + kStages * (((a_bytes + 1023) & ~1023) + ((b_bytes + 1023) & ~1023)) + kEpiStageBytes + kEpiSumFloats * 4 + (int)sizeof(TcShared) + 64;
    return true;
}

// act: bf16 [N,H,W,cin]; Wsrc: fp32 weights; transposed selects the dgrad pack
bool run_conv_tc(Exec &ex, const char *what, const void *act, Geom gin, int cin, int cout, int k, int stride,
                 const float *Wsrc, const bf16 *prepacked, bool transposed, Pair out, Pair partner, int sign, EpiReq req) {
    TcShape s;
    if (stride == 2 && (gin.H % 2 || gin.W % 2)) return false;
    const Geom g{gin.N, conv_out(gin.H, k, stride), conv_out(gin.W, k, stride)};   // output geometry
    if (!tc_shape(g, cin, cout, k, stride, s)) return false;
    const int taps = k * k;
    const int rows_pad = s.n_tiles * s.BN;
    if (!ex.dry && !encoder(ex.ctx)) return false;
    ex.flops += 2ull * g.P() * cout * cin * taps;
    int occ = (227 * 1024) / s.smem; if (occ > 2) occ = 2; if (occ < 1) occ = 1;
    int ctas = ex.ctx->sm_count * occ / s.n_tiles; if (ctas < 1) ctas = 1;
    if (ctas > s.g.n_px_tiles) ctas = s.g.n_px_tiles;
    size_t m = ex.ws.mark();
    bf16 *wp = prepacked ? const_cast<bf16 *>(prepacked) : ex.ws.get<bf16>((size_t)rows_pad * taps * s.cin_pad);
    const bool reduce = req.stats || req.bnbwd;
    float *part = reduce ? ex.ws.get<float>((size_t)ctas * 2 * cout) : nullptr;
    if (req.stats) req.stats->valid = true;
    if (!ex.dry) {
        EncodeTiledFn enc = encoder(ex.ctx);
        // without a pack made earlier in the step, build it from the fp32 master weights now
        if (!prepacked) {
            const size_t n = (size_t)rows_pad * taps * s.cin_pad;
            int grid = (int)((n + 255) / 256); if (grid > ex.ctx->sm_count * 4) grid = ex.ctx->sm_count * 4;
            if (!transposed) launch(ex, pack_weights_kernel, grid, 256, 0, Wsrc, wp, cout, cin, k, rows_pad, s.cin_pad, 0);
            else launch(ex, pack_weights_kernel, grid, 256, 0, Wsrc, wp, cin, cout, k, rows_pad, s.cin_pad, 1);
            ex.check("pack_weights", (double)n * 6);
        }
        CUtensorMap map_a, map_b;
        const CUtensorMapSwizzle sw = s.KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (s.KC == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
        {
            // the box spans stride x the tile in the input image and is walked with that stride
            cuuint64_t dims[4] = {(cuuint64_t)cin, (cuuint64_t)gin.W, (cuuint64_t)gin.H, (cuuint64_t)gin.N};
            cuuint64_t strides[3] = {(cuuint64_t)cin * 2, (cuuint64_t)gin.W * cin * 2, (cuuint64_t)gin.H * gin.W * cin * 2};
            cuuint32_t box[4] = {(cuuint32_t)s.KC, (cuuint32_t)(g.W * stride), (cuuint32_t)(s.g.BH * stride), (cuuint32_t)s.g.BIMG};
            cuuint32_t es[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
            CUresult r = enc(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, (void *)act, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) { ex.failed = true; ex.ctx->err = std::string(what) + ": tensor map (activations) rejected"; ex.ws.release(m); return true; }
        }
        {
            cuuint64_t dims[2] = {(cuuint64_t)taps * s.cin_pad, (cuuint64_t)rows_pad};
            cuuint64_t strides[1] = {(cuuint64_t)taps * s.cin_pad * 2};
            cuuint32_t box[2] = {(cuuint32_t)s.KC, (cuuint32_t)s.BN};
            cuuint32_t es[2] = {1, 1};
            CUresult r = enc(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void *)wp, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) { ex.failed = true; ex.ctx->err = std::string(what) + ": tensor map (weights) rejected"; ex.ws.release(m); return true; }
        }
        TcParams p;
        p.taps = taps; p.k = k; p.chunks = s.chunks; p.KC = s.KC; p.cin_pad = s.cin_pad; p.BN = s.BN; p.stride = stride; p.g = s.g;
        p.status = ex.ctx->dev_status;
        EpiArgs &e = p.epi;
        memset(&e, 0, sizeof e);
        e.mode = req.bnbwd ? EPI_BNBWD : (sign ? EPI_COUPLE : EPI_PLAIN);
        e.out = out; e.partner = partner; e.sign = sign; e.n_cols = cout; e.pitch = kEpiPitch;
        e.part = part; e.counter = reduce ? ex.ctx->counter() : nullptr;
        e.inv_count = 1.0 / (double)g.P(); e.eps = ex.eps;
        if (req.stats) { e.mean = req.stats->mean; e.rstd = req.stats->rstd; }
        if (req.bnbwd) { e.t = req.bnbwd->t; e.bn = req.bnbwd->bn; e.dgamma = req.bnbwd->dgamma; e.dbeta = req.bnbwd->dbeta; e.coef = req.bnbwd->coef; }
        static bool attr_set = false;
        if (!attr_set) { cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024); attr_set = true; }
        dim3 grid((unsigned)ctas, (unsigned)s.n_tiles);
        launch(ex, conv_tc_kernel, grid, kThreads, s.smem, map_a, map_b, p);
        const double bytes = (double)gin.P() * cin * 2 + (double)g.P() * cout * (sign || req.bnbwd ? 8 : 4) + (double)cout * taps * cin * 2;
        ex.check(what, bytes, 2.0 * g.P() * cout * cin * taps);
    }
    ex.ws.release(m);
    return true;
}

// ------------------------------------------------------------------------------------------------
// Weight gradient:  dW[co, tap, ci] = sum_p g[p, co] * a[p (+) tap, ci]
// GEMM view: the reduction runs over pixels.  Both operands are pixel-major in memory, so the tiles
// TMA delivers ([128 pixels][channel block]) are MN-major operands as they stand.  The M side
// stacks (tap, input-channel block) tiles -- one shifted TMA box each -- 128 rows per MMA group;
// the N side is a block of output channels.  A CTA owns up to two M groups and one N tile, walks
// its share of the pixel tiles (split-K) accumulating in tensor memory, and writes an fp32
// partial; the partials are summed in fixed order by splitk_sum_batch_kernel.
// For 3x3 layers of few channels the taps are split between the operands instead (sep):
//   dW[co, (kh, kw), ci] = sum_p a[p + (kh, 0), ci] * g[p - (0, kw), co]
// so the M side stacks the three vertical shifts of the activations, the N side the three horizontal
// shifts of the gradient: six boxes and one MMA group per pixel tile where the stacked form takes ten
// boxes and two groups.  (Activations outside the image are zero, so pixels p outside it add nothing.)
struct WgParams {
    int taps, k;
    int blockC, cblks, cin;      // input-channel block (16/32/64), blocks per tap, valid channels
    int total_blocks;            // taps * cblks
    int blockN, BN, cout;        // output-channel block, N tile, valid channels
    int GM;                      // M groups per CTA (1 or 2)
    int H, W, BH, BIMG;          // output geometry and tile
    int tiles_per_img, box_px;   // tiles per image (BIMG == 1); pixels a tile really holds (<= 128, the rest of its rows stay zero)
    int stride;
    int n_tiles_px;              // pixel tiles in all
    int stages;
    float *partial;              // splits > 1: [splits][taps][cin][cout], summed and transposed afterwards; else the gradient itself
    size_t slice;                // cout*taps*cin
    int *status;
    int a_region;                // bytes of a stage that hold activation blocks (the gradient blocks follow)
    int sep, cout_pad;           // sep: taps split between the operands (see the kernel); cout rounded up to 16
    int splits, m_chunks;        // this job's CTAs: split x M chunk x N tile, split fastest
    int cta0;                    // first CTA of the job in the launch
};

// One launch computes the weight gradients of up to kWgMaxJobs layers: each CTA finds its job from
// its index and then works on that layer alone.
constexpr int kWgMaxJobs = 4;
struct alignas(64) WgJob { CUtensorMap map_a, map_g; WgParams p; };
struct WgBatch { WgJob job[kWgMaxJobs]; int n; };

__global__ void __launch_bounds__(kThreads, 1)
wgrad_tc_kernel(const __grid_constant__ WgBatch batch) {
    int jb = 0;
    while (jb + 1 < batch.n && (int)blockIdx.x >= batch.job[jb + 1].p.cta0) jb++;
    const WgParams &p = batch.job[jb].p;
    const CUtensorMap &map_a = batch.job[jb].map_a, &map_g = batch.job[jb].map_g;
    const int local = (int)blockIdx.x - p.cta0;
    const int split = local % p.splits, chunk = (local / p.splits) % p.m_chunks, ntile = local / (p.splits * p.m_chunks);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int blk_bytes_a = 256 * p.blockC, blk_bytes_b = 256 * p.blockN;   // [128 pixels][block] bf16
    // a stage holds only the blocks a CTA really loads.  An M group is 128 rows = 32 KB from its first block:
    // the MMAs of a group that is not full read on into what follows (their rows of the result are never
    // stored), so the launch reserves room behind the last stage for that.
    const int a_region = p.a_region;
    const int stage_bytes = a_region + ((256 * p.BN + 1023) & ~1023);
    TcShared *sh = (TcShared *)(tiles + p.stages * stage_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bpg = 128 / p.blockC;                          // blocks per M group
    const int first_block = chunk * p.GM * bpg;
    int n_blocks = p.total_blocks - first_block; if (n_blocks > p.GM * bpg) n_blocks = p.GM * bpg;
    const int groups = (n_blocks + bpg - 1) / bpg;
    const int col0 = ntile * p.BN;
    int nb_n = (p.cout - col0 + p.blockN - 1) / p.blockN; if (nb_n > p.BN / p.blockN) nb_n = p.BN / p.blockN;   // N blocks holding valid channels
    const int npk = p.cout_pad / p.blockN;                   // sep: N blocks per horizontal shift
    if (p.sep) nb_n = p.k * npk;
    const int my_tiles = (p.n_tiles_px - split + p.splits - 1) / p.splits;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < p.GM * p.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; s++) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        mbar_init(&sh->acc_full[0], 1);
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&sh->tmem_base, tmem_cols);
    if (p.box_px < 128) {
        // a tile holds fewer than 128 pixels: the rows TMA never writes must not add to the pixel sum
        uint4 *z = reinterpret_cast<uint4 *>(tiles);
        const int n16 = p.stages * stage_bytes / 16;
        for (int i = threadIdx.x; i < n16; i += kThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
        fence_proxy_async();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    pdl_enter();             // the set-up above may overlap the kernel before; its outputs are read from here on
    const uint32_t tmem_d = sh->tmem_base;
    const int pad = p.k / 2;
    const int tiles_per_img = p.tiles_per_img;

    if (warp == 0) {
        // producer warp: lane 0 waits for the slot and arms the barrier, then every lane issues one box
        // (lane b < n_blocks: shifted activation block b; the next nb_n lanes: gradient blocks), so that
        // the loads of a tile leave in one instruction instead of one after the other
        const uint32_t tx = (uint32_t)(p.box_px * 2 * (n_blocks * p.blockC + nb_n * p.blockN));
        const bool a_lane = lane < n_blocks, g_lane = !a_lane && lane < n_blocks + nb_n;
        const int gb = first_block + lane, tap = gb / p.cblks, cb = gb - tap * p.cblks;
        const int kh = p.sep ? tap : tap / p.k, kw = p.sep ? p.k / 2 : tap - (tap / p.k) * p.k;
        const int bg = lane - n_blocks;
        const int g_c = p.sep ? (bg % npk) * p.blockN : col0 + bg * p.blockN;      // gradient box: first channel, first column
        const int g_x = p.sep ? p.k / 2 - bg / npk : 0;
        for (int it = 0; it < my_tiles; it++) {
            const int s = it % p.stages, round = it / p.stages;
            bool ok = true;
            if (lane == 0) {
                if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; }
                if (ok) mbar_expect_tx(&sh->full[s], tx);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const int t = split + it * p.splits;
            const int n0 = p.BIMG > 1 ? t * p.BIMG : t / tiles_per_img;
            const int h0 = p.BIMG > 1 ? 0 : (t % tiles_per_img) * p.BH;
            uint8_t *sa = tiles + s * stage_bytes;
            if (a_lane) tma_load_4d(sa + lane * blk_bytes_a, &map_a, &sh->full[s], cb * p.blockC, kw - pad, h0 * p.stride + kh - pad, n0);
            else if (g_lane) tma_load_4d(sa + a_region + bg * blk_bytes_b, &map_g, &sh->full[s], g_c, g_x, h0, n0);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(p.BN, true);
            const int rba = p.blockC * 2, rbb = p.blockN * 2;
            for (int it = 0; it < my_tiles; it++) {
                const int s = it % p.stages, round = it / p.stages;
                if (!mbar_wait(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = smem_u32(tiles + s * stage_bytes);
                for (int g = 0; g < groups; g++)
                    for (int ks = 0; ks < 8; ks++) {         // 16 pixels per MMA
                        const uint64_t da = smem_desc_mn(sa + g * 32768 + ks * 16 * rba, rba, blk_bytes_a);
                        const uint64_t db = smem_desc_mn(sa + a_region + ks * 16 * rbb, rbb, blk_bytes_b);
                        mma_bf16(tmem_d + (uint32_t)(g * p.BN), da, db, idesc, (it > 0 || ks > 0) ? 1u : 0u);
                    }
                mma_commit(&sh->empty[s]);
            }
            mma_commit(&sh->acc_full[0]);
        }
    } else {
        const int quarter = warp & 3;
        bool ok = true;
        if (quarter == 0 && lane == 0) ok = mbar_wait(&sh->acc_full[0], 0);     // one thread polls, the rest block
        ok = named_barrier_and(2, 128, ok);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok && sh->failed == 0) {
            const int m = quarter * 32 + lane;
            float *dst = p.partial + (size_t)split * p.slice;
            for (int g = 0; g < groups; g++) {
                const int gb = first_block + g * bpg + m / p.blockC;
                const int tap_m = gb / p.cblks, ci = (gb - tap_m * p.cblks) * p.blockC + m % p.blockC;     // sep: tap_m is kh
                const bool row_ok = gb < p.total_blocks && ci < p.cin;
                for (int c = 0; c < p.BN; c += 16) {
                    float v[16];
                    tmem_ld16(tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(g * p.BN + c), v);   // whole warp takes part
                    if (!row_ok) continue;
                    if (my_tiles == 0) {
#pragma unroll
                        for (int j = 0; j < 16; j++) v[j] = 0.f;
                    }
                    // column c of the accumulator: output channel cb0 + ..., and with sep the horizontal shift too
                    const int kw = p.sep ? c / p.cout_pad : 0;
                    const int cb0 = p.sep ? c - kw * p.cout_pad : col0 + c;
                    const int tap = p.sep ? tap_m * p.k + kw : tap_m;
                    if (p.splits > 1) {
                        // split partials are [tap][ci][co]: this row's output channels are contiguous (cout is a multiple of 8)
                        float *row = dst + ((size_t)tap * p.cin + ci) * p.cout + cb0;
#pragma unroll
                        for (int j = 0; j < 16; j += 4)
                            if (cb0 + j < p.cout) *reinterpret_cast<float4 *>(row + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; j++) {
                            const int co = cb0 + j;
                            if (co < p.cout) dst[((size_t)co * p.taps + tap) * p.cin + ci] = v[j];
                        }
                    }
                }
            }
        } else if (lane == 0) {
            atomicExch(&sh->failed, 1u);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && sh->failed) atomicExch(p.status, (int)REVNET_E_TIMEOUT);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(tmem_cols) : "memory");
    }
}

// dW[co][tap][ci] = sum over splits of part[z][tap][ci][co], in a fixed order: 8 interleaved groups of
// splits per element, combined through shared memory (256 threads = 32 elements x 8 groups); several
// (partials, destination) pairs in one launch, blockIdx.y picks the pair
struct SumBatch { const float *part[kWgMaxJobs]; float *out[kWgMaxJobs]; size_t n[kWgMaxJobs]; int splits[kWgMaxJobs], cout[kWgMaxJobs], rows[kWgMaxJobs]; };
__global__ void splitk_sum_batch_kernel(const SumBatch b) {
    pdl_enter();
    __shared__ float sm[8][33];
    const int j = blockIdx.y;
    const float *__restrict__ part = b.part[j];
    const size_t n = b.n[j];
    const int splits = b.splits[j];
    const int e = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const size_t i = (size_t)blockIdx.x * 32 + e;
    float s = 0.f;
    if (i < n)
        for (int z = grp; z < splits; z += 8) s += part[(size_t)z * n + i];
    sm[grp][e] = s;
    __syncthreads();
    if (grp == 0 && i < n) {
        for (int g = 1; g < 8; g++) s += sm[g][e];
        const size_t row = i / (size_t)b.cout[j];              // (tap, ci)
        const int co = (int)(i - row * (size_t)b.cout[j]);
        b.out[j][(size_t)co * b.rows[j] + row] = s;
    }
}

int pick_block(int c_pad) { return c_pad % 64 == 0 ? 64 : (c_pad % 32 == 0 ? 32 : 16); }

// g: geometry of the tensor; (tile_w, BH, BIMG): the 128-pixel tile in units of the traversal stride
bool encode_act_map(Exec &ex, CUtensorMap *map, const void *base, Geom g, int C, int box_c, int tile_w, int BH, int BIMG, int stride) {
    const CUtensorMapSwizzle sw = box_c == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (box_c == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N};
    cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)g.W * C * 2, (cuuint64_t)g.H * g.W * C * 2};
    cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)(tile_w * stride), (cuuint32_t)(BH * stride), (cuuint32_t)BIMG};
    cuuint32_t es[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    return encoder(ex.ctx)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, (void *)base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool conv_fprop_tc(Exec &ex, const void *a, Geom gi, const Layer &L, Pair out, Pair partner, int sign, Moments *stats) {
    EpiReq req; req.stats = stats;
    return run_conv_tc(ex, "conv_fprop_tc", a, gi, L.cin, L.cout, L.k, L.stride, L.W, L.Wp_fprop, false, out, partner, sign, req);
}

// da[q,ci] = sum_{tap,co} g[q (-) tap, co] W[co,tap,ci]: a stride-1 convolution of g with the mirrored, transposed weights
bool conv_dgrad_tc(Exec &ex, const void *g, Geom gi, const Layer &L, float *da, const BnBwdReq *bb) {
    if (L.stride != 1) return false;
    EpiReq req; req.bnbwd = bb;
    return run_conv_tc(ex, "conv_dgrad_tc", g, gi, L.cout, L.cin, L.k, L.stride, L.W, L.Wp_dgrad, true, single(da, L.cin), Pair{}, 0, req);
}


constexpr int kWgSmemMax = 224 * 1024;

// Shape decisions of one layer's weight gradient; cta_budget: the CTAs the job may take
struct WgPlan { WgParams p; Geom go; int n_tiles, stage_bytes, tail_bytes; };
static bool wgrad_plan(Geom gi, const Layer &L, int cta_budget, WgPlan &w, bool allow_sep = true) {
    if ((L.stride != 1 && L.stride != 2) || (L.k != 1 && L.k != 3) || L.cin % 8 || L.cout % 8) return false;
    if (L.stride == 2 && (gi.H % 2 || gi.W % 2)) return false;
    WgParams &p = w.p;
    w.go = Geom{gi.N, conv_out(gi.H, L.k, L.stride), conv_out(gi.W, L.k, L.stride)};   // tiles walk the output pixels
    TileGeom tg;
    if (!tile_geom(w.go, tg) || tg.W * L.stride > 256 || tg.BH * L.stride > 256) return false;
    p.BH = tg.BH; p.BIMG = tg.BIMG; p.tiles_per_img = tg.tiles_per_img; p.box_px = tg.BIMG * tg.BH * tg.W;
    const int taps = L.k * L.k, cin_pad = round_up(L.cin, 16), cout_pad = round_up(L.cout, 16);
    p.taps = taps; p.k = L.k; p.cin = L.cin; p.cout = L.cout;
    p.blockC = pick_block(cin_pad); p.cblks = cin_pad / p.blockC;
    p.blockN = pick_block(cout_pad);
    p.cout_pad = cout_pad;
    const int bpg = 128 / p.blockC;
    // taps split between the operands when the three shifted activation blocks fit one M group, the three
    // shifted gradient blocks one N tile, and the boxes of a pixel tile the lanes of the producer warp
    p.sep = (allow_sep && L.k == 3 && L.stride == 1 && 3 * cin_pad <= 128 && 3 * cout_pad <= 256 && 2 * bpg + 3 * (cout_pad / p.blockN) <= 32) ? 1 : 0;
    if (p.sep) {
        p.total_blocks = L.k * p.cblks;
        p.BN = L.k * cout_pad;
    } else {
        p.total_blocks = taps * p.cblks;
        p.BN = cout_pad <= 128 ? cout_pad : 128;
        if (p.BN % p.blockN) p.BN = p.blockN;
    }
    const int groups_all = (p.total_blocks + bpg - 1) / bpg;
    p.GM = groups_all >= 2 ? 2 : 1;
    p.m_chunks = (groups_all + p.GM - 1) / p.GM;
    w.n_tiles = p.sep ? 1 : (cout_pad + p.BN - 1) / p.BN;
    p.H = w.go.H; p.W = w.go.W; p.stride = L.stride;
    p.n_tiles_px = tg.n_px_tiles;
    const int blocks_max = p.total_blocks < p.GM * bpg ? p.total_blocks : p.GM * bpg;
    p.a_region = (blocks_max * 256 * p.blockC + 1023) & ~1023;
    w.stage_bytes = p.a_region + ((256 * p.BN + 1023) & ~1023);
    w.tail_bytes = p.GM * 32768 - p.a_region;        // what the MMAs of a partly filled group read past the last stage
    p.stages = (kWgSmemMax - 2048 - w.tail_bytes) / w.stage_bytes; if (p.stages > kStages) p.stages = kStages;
    if (p.stages < 2) return p.sep ? wgrad_plan(gi, L, cta_budget, w, false) : false;
    // split the pixel reduction so that the job's CTAs cover its share of the machine once
    int splits = (cta_budget + p.m_chunks * w.n_tiles - 1) / (p.m_chunks * w.n_tiles);
    if (splits > p.n_tiles_px) splits = p.n_tiles_px;
    if (splits < 1) splits = 1;
    p.splits = splits;
    p.slice = (size_t)L.cout * taps * L.cin;
    return true;
}

// Weight gradients of n layers (n <= 4) in one launch, and one more launch that sums their split partials.
// scratch: room for the split partials if the caller provides it (else it comes from the arena);
// need: if non-null the call only reports whether it takes the shapes and how many floats of scratch it wants
bool conv_wgrad_tc_batch(Exec &ex, int n, const void *const *gq, const void *const *a, const Geom *gi, const Layer *const *L,
                         float *scratch, size_t *need) {
    if (n < 1 || n > kWgMaxJobs) return false;
    WgPlan w[kWgMaxJobs];
    const int budget = ex.ctx->sm_count / n;
    size_t total = 0;
    for (int j = 0; j < n; j++) {
        if (!wgrad_plan(gi[j], *L[j], budget, w[j])) return false;
        if (w[j].p.splits > 1) total += (size_t)w[j].p.splits * w[j].p.slice;
    }
    if (need) { *need = total; return true; }
    if (!ex.dry && !encoder(ex.ctx)) return false;
    size_t m = ex.ws.mark();
    float *part = total ? (scratch ? scratch : ex.ws.get<float>(total)) : nullptr;
    for (int j = 0; j < n; j++) ex.flops += 2ull * w[j].go.P() * L[j]->cout * L[j]->cin * w[j].p.taps;
    if (!ex.dry) {
        WgBatch batch;
        SumBatch sums;
        batch.n = n;
        int cta = 0, smem = 0, n_sums = 0;
        size_t off = 0, max_slice = 0;
        double bytes = 0, flops = 0, sum_bytes = 0;
        for (int j = 0; j < n; j++) {
            WgParams &p = w[j].p;
            if (!encode_act_map(ex, &batch.job[j].map_a, a[j], gi[j], L[j]->cin, p.blockC, w[j].go.W, p.BH, p.BIMG, L[j]->stride) ||
                !encode_act_map(ex, &batch.job[j].map_g, gq[j], w[j].go, L[j]->cout, p.blockN, w[j].go.W, p.BH, p.BIMG, 1)) {
                ex.failed = true; ex.ctx->err = "conv_wgrad_tc: tensor map rejected"; ex.ws.release(m); return true;
            }
            p.status = ex.ctx->dev_status;
            p.cta0 = cta;
            cta += p.splits * p.m_chunks * w[j].n_tiles;
            if (p.splits > 1) {
                p.partial = part + off;
                sums.part[n_sums] = p.partial; sums.out[n_sums] = L[j]->dW; sums.n[n_sums] = p.slice; sums.splits[n_sums] = p.splits;
                sums.cout[n_sums] = L[j]->cout; sums.rows[n_sums] = p.taps * L[j]->cin;
                n_sums++;
                off += (size_t)p.splits * p.slice;
                if (p.slice > max_slice) max_slice = p.slice;
                sum_bytes += (double)p.slice * 4 * (p.splits + 1);
            } else {
                p.partial = L[j]->dW;
            }
            batch.job[j].p = p;
            const int sm = 1024 + p.stages * w[j].stage_bytes + w[j].tail_bytes + (int)sizeof(TcShared) + 64;
            if (sm > smem) smem = sm;
            bytes += (double)gi[j].P() * L[j]->cin * 2 + (double)w[j].go.P() * L[j]->cout * 2 + (double)p.slice * 4 * p.splits;
            flops += 2.0 * w[j].go.P() * L[j]->cout * L[j]->cin * p.taps;
        }
        static bool attr_set = false;
        if (!attr_set) { cudaFuncSetAttribute(wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kWgSmemMax); attr_set = true; }
        launch(ex, wgrad_tc_kernel, (unsigned)cta, kThreads, smem, batch);
        ex.check("conv_wgrad_tc", bytes, flops);
        if (n_sums) {
            dim3 grid((unsigned)((max_slice + 31) / 32), (unsigned)n_sums);
            launch(ex, splitk_sum_batch_kernel, grid, 256, 0, sums);
            ex.check("splitk_sum", sum_bytes);
        }
    }
    ex.ws.release(m);
    return true;
}

bool conv_wgrad_tc(Exec &ex, const void *gq, const void *a, Geom gi, const Layer &L, float *dW, float *scratch, size_t *need) {
    Layer one = L;
    one.dW = dW;
    const Layer *lp = &one;
    return conv_wgrad_tc_batch(ex, 1, &gq, &a, &gi, &lp, scratch, need);
}

void *tc_encoder(revnet_ctx *ctx) { return (void *)encoder(ctx); }

// pack of one layer built on the spot (calls that have no step-level pack)
void tc_pack_now(Exec &ex, const float *W, bf16 *out, int cin, int cout, int k, bool transposed) {
    if (ex.dry) return;
    const PackJob j = tc_pack_job(W, out, cin, cout, k, transposed);
    const size_t n = (size_t)j.rows_pad * k * k * j.cols_pad;
    int grid = (int)((n + 255) / 256); if (grid > ex.ctx->sm_count * 4) grid = ex.ctx->sm_count * 4;
    launch(ex, pack_weights_kernel, grid, 256, 0, W, out, cout, cin, k, j.rows_pad, j.cols_pad, transposed ? 1 : 0);
    ex.check("pack_weights", (double)n * 6);
}

// ---- packs made once per step (the train step calls these before the forward pass)
static void pack_dims(int rows, int cols, int &rows_pad, int &cols_pad) {
    const int rp = round_up(rows, 16), BN = rp <= 128 ? rp : 128;
    rows_pad = (rp + BN - 1) / BN * BN;
    cols_pad = round_up(cols, 16);
}
size_t tc_pack_elems(int cin, int cout, int k, bool transposed) {
    int rp, cp;
    if (!transposed) pack_dims(cout, cin, rp, cp); else pack_dims(cin, cout, rp, cp);
    return (size_t)rp * k * k * cp;
}
PackJob tc_pack_job(const float *W, bf16 *out, int cin, int cout, int k, bool transposed) {
    PackJob j;
    j.W = W; j.out = out; j.Co = cout; j.Ci = cin; j.k = k; j.transposed = transposed ? 1 : 0;
    if (!transposed) pack_dims(cout, cin, j.rows_pad, j.cols_pad); else pack_dims(cin, cout, j.rows_pad, j.cols_pad);
    return j;
}
void tc_pack_batch(Exec &ex, const PackJob *jobs_dev, int n_jobs, double bytes, size_t max_job_elems) {
    if (ex.dry || n_jobs == 0) return;
    // blocks per job sized for the largest job (2048 elements per block), within 4 .. 96
    size_t bx = (max_job_elems + 2047) / 2048;
    if (bx < 4) bx = 4; if (bx > 96) bx = 96;
    dim3 grid((unsigned)bx, (unsigned)n_jobs);
    launch(ex, pack_weights_batch_kernel, grid, 256, 0, jobs_dev);
    ex.check("pack_weights_batch", bytes);
}
