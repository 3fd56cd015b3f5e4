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
#include <cuda.h>

namespace {

constexpr int kStages = 4;
constexpr int kThreads = 192;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s: far beyond any real wait of this kernel

struct TcParams {
    int taps;        // k*k
    int k;           // kernel size
    int chunks;      // channel chunks per tap
    int KC;          // channels per chunk (16, 32 or 64)
    int cin_pad;     // chunks * KC
    int BN;          // N tile
    int n_cols;      // valid output channels
    int H, W;        // output image size
    int stride;      // 1 or 2: input pixel = output pixel * stride + tap - pad (TMA traversal stride)
    int BH, BIMG;    // tile: BH rows x W columns x BIMG images = 128 pixels
    Pair out, partner;
    int sign;
    int *status;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// bounded wait: false when the limit ran out
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; it++) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if ((it & 63) == 63) {
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) return false;
        }
    }
}

__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

// shared-memory matrix descriptor, K-major operand whose rows are `row_bytes` (32/64/128) long and
// stored with the matching TMA swizzle; 8-row groups are row_bytes*8 apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, int row_bytes) {
    const uint64_t layout = row_bytes == 128 ? 2 : (row_bytes == 64 ? 4 : 6);
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);                 // start address
    d |= (uint64_t)1 << 16;                                 // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)((row_bytes * 8) >> 4) << 32;            // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                                 // descriptor version
    d |= layout << 61;
    return d;
}

// instruction descriptor: bf16 x bf16 -> fp32, M = 128; mn_major: both operands have their M / N
// index contiguous in shared memory (pixel-major tiles of the weight-gradient GEMM), else K-major
__device__ __forceinline__ uint32_t instr_desc(int n, bool mn_major = false) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (mn_major ? (3u << 15) : 0u) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// descriptor of an MN-major operand: rows are K indices, each row holds `row_bytes` (32/64/128) of
// contiguous M (or N) elements with the matching swizzle; the next block of M / N elements starts
// `block_bytes` further on, groups of 8 K-rows are row_bytes*8 apart
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, int row_bytes, int block_bytes) {
    const uint64_t layout = row_bytes == 128 ? 2 : (row_bytes == 64 ? 4 : 6);
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((block_bytes >> 4) & 0x3FFF) << 16;     // leading byte offset: between M / N blocks
    d |= (uint64_t)((row_bytes * 8) >> 4) << 32;            // stride byte offset: between 8-row K groups
    d |= (uint64_t)1 << 46;
    d |= layout << 61;
    return d;
}

__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; i++) v[i] = __uint_as_float(r[i]);
}

struct __align__(8) TcShared {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t acc_full;
    uint32_t tmem_base;
    uint32_t failed;
};

__global__ void __launch_bounds__(kThreads, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // operand stages first (1024-byte aligned for the 128-byte swizzle), bookkeeping behind them
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int a_bytes = 128 * p.KC * 2, b_bytes = p.BN * p.KC * 2;
    const int b_off = (a_bytes + 1023) & ~1023;
    const int stage_bytes = b_off + ((b_bytes + 1023) & ~1023);
    TcShared *sh = (TcShared *)(tiles + kStages * stage_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int iters = p.taps * p.chunks;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < p.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; s++) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        mbar_init(&sh->acc_full, 1);
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = sh->tmem_base;

    // tile origin: tiles are runs of 128 consecutive pixels in (n, h, w) order
    const int tiles_per_img = p.BIMG > 1 ? 1 : p.H / p.BH;
    const int n0 = p.BIMG > 1 ? blockIdx.x * p.BIMG : blockIdx.x / tiles_per_img;
    const int h0 = p.BIMG > 1 ? 0 : (blockIdx.x % tiles_per_img) * p.BH;
    const int col0 = blockIdx.y * p.BN;
    const int pad = p.k / 2;

    if (warp == 0) {
        if (lane == 0) {
            for (int it = 0; it < iters; it++) {
                const int s = it % kStages, round = it / kStages;
                if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); break; }
                const int tap = it / p.chunks, ch = it - tap * p.chunks;
                const int kh = tap / p.k, kw = tap - kh * p.k;
                uint8_t *sa = tiles + s * stage_bytes;
                mbar_expect_tx(&sh->full[s], (uint32_t)(a_bytes + b_bytes));
                tma_load_4d(sa, &map_a, &sh->full[s], ch * p.KC, kw - pad, h0 * p.stride + kh - pad, n0);
                tma_load_2d(sa + b_off, &map_b, &sh->full[s], tap * p.cin_pad + ch * p.KC, col0);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(p.BN);
            const int row_bytes = p.KC * 2;
            bool ok = true;
            for (int it = 0; it < iters && ok; it++) {
                const int s = it % kStages, round = it / kStages;
                if (!mbar_wait(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = smem_u32(tiles + s * stage_bytes);
                for (int kk = 0; kk < p.KC / 16; kk++) {
                    const uint64_t da = smem_desc(sa + kk * 32, row_bytes);
                    const uint64_t db = smem_desc(sa + b_off + kk * 32, row_bytes);
                    mma_bf16(tmem_d, da, db, idesc, (it > 0 || kk > 0) ? 1u : 0u);
                }
                mma_commit(&sh->empty[s]);          // frees the stage once these MMAs have read it
            }
            mma_commit(&sh->acc_full);              // accumulator complete (also issued after a failure, so nobody waits forever)
        }
    } else {
        // epilogue: warp w owns accumulator lanes 32*(w%4) .. +31 = pixel rows of the tile
        const int quarter = warp & 3;
        const bool ok = mbar_wait(&sh->acc_full, 0);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok && sh->failed == 0) {
            const size_t row = (size_t)blockIdx.x * 128 + quarter * 32 + lane;
            for (int c = 0; c < p.BN; c += 16) {
                float v[16];
                tmem_ld16(tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, v);
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    const int col = col0 + c + j;
                    if (col < p.n_cols) p.out.couple4(row, col, make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]), p.partner, p.sign);
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

// ---- weight packs: bf16 [rows_pad][taps][cin_pad]; transposed = true builds the dgrad operand
// (rows = input channels, columns = output channels, taps mirrored)
__global__ void pack_weights_kernel(const float *__restrict__ W, bf16 *__restrict__ out, int Co, int Ci, int k,
                                    int rows_pad, int cols_pad, int transposed) {
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

struct TcShape { int KC, cin_pad, chunks, BN, n_tiles, BH, BIMG, smem; };

// Which shapes the kernel takes: stride 1 or 2, k in {1,3}; a 128-pixel output tile must be whole rows of one
// image or whole images; channel rows 16-byte aligned for TMA.
bool tc_shape(Geom g, int cin, int cout, int k, int stride, TcShape &s) {   // g: output geometry
    if ((stride != 1 && stride != 2) || (k != 1 && k != 3) || cin % 8 || cout % 4) return false;
    const int W = g.W, H = g.H;
    if (W > 128 || 128 % W) return false;
    if (H * W >= 128) { if (H % (128 / W)) return false; s.BH = 128 / W; s.BIMG = 1; }
    else { if (128 % (H * W) || g.N % (128 / (H * W))) return false; s.BH = H; s.BIMG = 128 / (H * W); }
    s.cin_pad = round_up(cin, 16);
    s.KC = s.cin_pad % 64 == 0 ? 64 : (s.cin_pad % 32 == 0 ? 32 : 16);
    s.chunks = s.cin_pad / s.KC;
    const int cout_pad = round_up(cout, 16);
    s.BN = cout_pad <= 128 ? cout_pad : 128;
    s.n_tiles = (cout_pad + s.BN - 1) / s.BN;
    const int a_bytes = 128 * s.KC * 2, b_bytes = s.BN * s.KC * 2;
    s.smem = 1024 + kStages * (((a_bytes + 1023) & ~1023) + ((b_bytes + 1023) & ~1023)) + (int)sizeof(TcShared) + 64;
    return true;
}

// act: bf16 [N,H,W,cin]; Wsrc: fp32 weights; transposed selects the dgrad pack
bool run_conv_tc(Exec &ex, const char *what, const void *act, Geom gin, int cin, int cout, int k, int stride,
                 const float *Wsrc, const bf16 *prepacked, bool transposed, Pair out, Pair partner, int sign) {
    TcShape s;
    if (stride == 2 && (gin.H % 2 || gin.W % 2)) return false;
    const Geom g{gin.N, conv_out(gin.H, k, stride), conv_out(gin.W, k, stride)};   // output geometry
    if (!tc_shape(g, cin, cout, k, stride, s)) return false;
    const int taps = k * k, cout_pad = round_up(cout, 16);
    const int rows_pad = s.n_tiles * s.BN;
    if (!ex.dry && !encoder(ex.ctx)) return false;
    ex.flops += 2ull * g.P() * cout * cin * taps;
    size_t m = ex.ws.mark();
    bf16 *wp = prepacked ? const_cast<bf16 *>(prepacked) : ex.ws.get<bf16>((size_t)rows_pad * taps * s.cin_pad);
    (void)cout_pad;
    if (!ex.dry) {
        EncodeTiledFn enc = encoder(ex.ctx);
        // without a pack made earlier in the step, build it from the fp32 master weights now
        if (!prepacked) {
            const size_t n = (size_t)rows_pad * taps * s.cin_pad;
            int grid = (int)((n + 255) / 256); if (grid > ex.ctx->sm_count * 4) grid = ex.ctx->sm_count * 4;
            if (!transposed) pack_weights_kernel<<<grid, 256, 0, ex.stream>>>(Wsrc, wp, cout, cin, k, rows_pad, s.cin_pad, 0);
            else pack_weights_kernel<<<grid, 256, 0, ex.stream>>>(Wsrc, wp, cin, cout, k, rows_pad, s.cin_pad, 1);
            ex.check("pack_weights", (double)n * 6);
        }
        CUtensorMap map_a, map_b;
        const CUtensorMapSwizzle sw = s.KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (s.KC == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
        {
            // the box spans stride x the tile in the input image and is walked with that stride
            cuuint64_t dims[4] = {(cuuint64_t)cin, (cuuint64_t)gin.W, (cuuint64_t)gin.H, (cuuint64_t)gin.N};
            cuuint64_t strides[3] = {(cuuint64_t)cin * 2, (cuuint64_t)gin.W * cin * 2, (cuuint64_t)gin.H * gin.W * cin * 2};
            cuuint32_t box[4] = {(cuuint32_t)s.KC, (cuuint32_t)(g.W * stride), (cuuint32_t)(s.BH * stride), (cuuint32_t)s.BIMG};
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
        p.taps = taps; p.k = k; p.chunks = s.chunks; p.KC = s.KC; p.cin_pad = s.cin_pad; p.BN = s.BN; p.n_cols = cout;
        p.H = g.H; p.W = g.W; p.stride = stride; p.BH = s.BH; p.BIMG = s.BIMG; p.out = out; p.partner = partner; p.sign = sign; p.status = ex.ctx->dev_status;
        static bool attr_set = false;
        if (!attr_set) { cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024); attr_set = true; }
        dim3 grid((unsigned)(g.P() / 128), (unsigned)s.n_tiles);
        conv_tc_kernel<<<grid, kThreads, s.smem, ex.stream>>>(map_a, map_b, p);
        const double bytes = (double)gin.P() * cin * 2 + (double)g.P() * cout * (sign ? 8 : 4) + (double)cout * taps * cin * 2;
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
// partial; the partials are summed in fixed order by splitk_sum_kernel.
struct WgParams {
    int taps, k;
    int blockC, cblks, cin;      // input-channel block (16/32/64), blocks per tap, valid channels
    int total_blocks;            // taps * cblks
    int blockN, BN, cout;        // output-channel block, N tile, valid channels
    int GM;                      // M groups per CTA (1 or 2)
    int H, W, BH, BIMG;          // output geometry and tile
    int stride;
    int n_tiles_px;              // pixel tiles in all
    int stages;
    float *partial;              // [splits][cout][taps][cin]
    size_t slice;                // cout*taps*cin
    int *status;
};

__global__ void __launch_bounds__(kThreads, 1)
wgrad_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_g, const WgParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int blk_bytes_a = 256 * p.blockC, blk_bytes_b = 256 * p.blockN;   // [128 pixels][block] bf16
    const int a_region = p.GM * 32768;                                       // 128 M rows x 128 pixels x 2 B per group
    const int stage_bytes = a_region + ((256 * p.BN + 1023) & ~1023);
    TcShared *sh = (TcShared *)(tiles + p.stages * stage_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bpg = 128 / p.blockC;                          // blocks per M group
    const int first_block = blockIdx.y * p.GM * bpg;
    int n_blocks = p.total_blocks - first_block; if (n_blocks > p.GM * bpg) n_blocks = p.GM * bpg;
    const int groups = (n_blocks + bpg - 1) / bpg;
    const int col0 = blockIdx.z * p.BN;
    int nb_n = (p.cout - col0 + p.blockN - 1) / p.blockN; if (nb_n > p.BN / p.blockN) nb_n = p.BN / p.blockN;   // N blocks holding valid channels
    const int my_tiles = (p.n_tiles_px - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < p.GM * p.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; s++) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        mbar_init(&sh->acc_full, 1);
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = sh->tmem_base;
    const int pad = p.k / 2;
    const int tiles_per_img = p.BIMG > 1 ? 1 : p.H / p.BH;

    if (warp == 0) {
        if (lane == 0) {
            const uint32_t tx = (uint32_t)(n_blocks * blk_bytes_a + nb_n * blk_bytes_b);
            for (int it = 0; it < my_tiles; it++) {
                const int s = it % p.stages, round = it / p.stages;
                if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); break; }
                const int t = blockIdx.x + it * gridDim.x;
                const int n0 = p.BIMG > 1 ? t * p.BIMG : t / tiles_per_img;
                const int h0 = p.BIMG > 1 ? 0 : (t % tiles_per_img) * p.BH;
                uint8_t *sa = tiles + s * stage_bytes;
                mbar_expect_tx(&sh->full[s], tx);
                for (int b = 0; b < n_blocks; b++) {
                    const int gb = first_block + b, tap = gb / p.cblks, cb = gb - tap * p.cblks;
                    const int kh = tap / p.k, kw = tap - kh * p.k;
                    tma_load_4d(sa + b * blk_bytes_a, &map_a, &sh->full[s], cb * p.blockC, kw - pad, h0 * p.stride + kh - pad, n0);
                }
                for (int b = 0; b < nb_n; b++)
                    tma_load_4d(sa + a_region + b * blk_bytes_b, &map_g, &sh->full[s], col0 + b * p.blockN, 0, h0, n0);
            }
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
            mma_commit(&sh->acc_full);
        }
    } else {
        const int quarter = warp & 3;
        const bool ok = mbar_wait(&sh->acc_full, 0);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok && sh->failed == 0) {
            const int m = quarter * 32 + lane;
            float *dst = p.partial + (size_t)blockIdx.x * p.slice;
            for (int g = 0; g < groups; g++) {
                const int gb = first_block + g * bpg + m / p.blockC;
                const int tap = gb / p.cblks, ci = (gb - tap * p.cblks) * p.blockC + m % p.blockC;
                const bool row_ok = gb < p.total_blocks && ci < p.cin;
                for (int c = 0; c < p.BN; c += 16) {
                    float v[16];
                    tmem_ld16(tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(g * p.BN + c), v);   // whole warp takes part
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 16; j++) {
                            const int co = col0 + c + j;
                            if (co < p.cout) dst[((size_t)co * p.taps + tap) * p.cin + ci] = my_tiles > 0 ? v[j] : 0.f;
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

// out[i] = sum over splits of part[z][i], in a fixed order: 8 interleaved groups of splits per
// element, combined through shared memory (256 threads = 32 elements x 8 groups)
__global__ void splitk_sum_kernel(const float *__restrict__ part, size_t n, int splits, float *__restrict__ out) {
    __shared__ float sm[8][33];
    const int e = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const size_t i = (size_t)blockIdx.x * 32 + e;
    float s = 0.f;
    if (i < n)
        for (int z = grp; z < splits; z += 8) s += part[(size_t)z * n + i];
    sm[grp][e] = s;
    __syncthreads();
    if (grp == 0 && i < n) {
        for (int g = 1; g < 8; g++) s += sm[g][e];
        out[i] = s;
    }
}

int pick_block(int c_pad) { return c_pad % 64 == 0 ? 64 : (c_pad % 32 == 0 ? 32 : 16); }

bool tile_shape(Geom g, int &BH, int &BIMG) {
    const int W = g.W, H = g.H;
    if (W > 128 || 128 % W) return false;
    if (H * W >= 128) { if (H % (128 / W)) return false; BH = 128 / W; BIMG = 1; }
    else { if (128 % (H * W) || g.N % (128 / (H * W))) return false; BH = H; BIMG = 128 / (H * W); }
    return true;
}

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

bool conv_fprop_tc(Exec &ex, const void *a, Geom gi, const Layer &L, Pair out, Pair partner, int sign) {
    return run_conv_tc(ex, "conv_fprop_tc", a, gi, L.cin, L.cout, L.k, L.stride, L.W, L.Wp_fprop, false, out, partner, sign);
}

// da[q,ci] = sum_{tap,co} g[q (-) tap, co] W[co,tap,ci]: a stride-1 convolution of g with the mirrored, transposed weights
bool conv_dgrad_tc(Exec &ex, const void *g, Geom gi, const Layer &L, float *da) {
    if (L.stride != 1) return false;
    return run_conv_tc(ex, "conv_dgrad_tc", g, gi, L.cout, L.cin, L.k, L.stride, L.W, L.Wp_dgrad, true, single(da, L.cin), Pair{}, 0);
}


bool conv_wgrad_tc(Exec &ex, const void *gq, const void *a, Geom gi, const Layer &L, float *dW) {
    if ((L.stride != 1 && L.stride != 2) || (L.k != 1 && L.k != 3) || L.cin % 8 || L.cout % 8) return false;
    if (L.stride == 2 && (gi.H % 2 || gi.W % 2)) return false;
    WgParams p;
    const Geom go{gi.N, conv_out(gi.H, L.k, L.stride), conv_out(gi.W, L.k, L.stride)};   // tiles walk the output pixels
    if (!tile_shape(go, p.BH, p.BIMG)) return false;
    if (!ex.dry && !encoder(ex.ctx)) return false;
    const int taps = L.k * L.k, cin_pad = round_up(L.cin, 16), cout_pad = round_up(L.cout, 16);
    p.taps = taps; p.k = L.k; p.cin = L.cin; p.cout = L.cout;
    p.blockC = pick_block(cin_pad); p.cblks = cin_pad / p.blockC; p.total_blocks = taps * p.cblks;
    p.blockN = pick_block(cout_pad);
    p.BN = cout_pad <= 128 ? cout_pad : 128;
    if (p.BN % p.blockN) p.BN = p.blockN;
    const int bpg = 128 / p.blockC;
    const int groups_all = (p.total_blocks + bpg - 1) / bpg;
    p.GM = groups_all >= 2 ? 2 : 1;
    const int m_chunks = (groups_all + p.GM - 1) / p.GM;
    const int n_tiles = (cout_pad + p.BN - 1) / p.BN;
    p.H = go.H; p.W = go.W; p.stride = L.stride;
    p.n_tiles_px = (int)(go.P() / 128);
    const int stage_bytes = p.GM * 32768 + ((256 * p.BN + 1023) & ~1023);
    p.stages = (200 * 1024 - 2048) / stage_bytes; if (p.stages > kStages) p.stages = kStages;
    if (p.stages < 2) return false;
    // split the pixel reduction so that the grid covers the machine once
    int splits = (ex.ctx->sm_count + m_chunks * n_tiles - 1) / (m_chunks * n_tiles);
    if (splits > p.n_tiles_px) splits = p.n_tiles_px;
    if (splits < 1) splits = 1;
    p.slice = (size_t)L.cout * taps * L.cin;
    ex.flops += 2ull * go.P() * L.cout * L.cin * taps;
    size_t m = ex.ws.mark();
    float *part = splits > 1 ? ex.ws.get<float>((size_t)splits * p.slice) : dW;
    if (!ex.dry) {
        CUtensorMap map_a, map_g;
        if (!encode_act_map(ex, &map_a, a, gi, L.cin, p.blockC, go.W, p.BH, p.BIMG, L.stride) ||
            !encode_act_map(ex, &map_g, gq, go, L.cout, p.blockN, go.W, p.BH, p.BIMG, 1)) {
            ex.failed = true; ex.ctx->err = "conv_wgrad_tc: tensor map rejected"; ex.ws.release(m); return true;
        }
        p.partial = part; p.status = ex.ctx->dev_status;
        static bool attr_set = false;
        if (!attr_set) { cudaFuncSetAttribute(wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024); attr_set = true; }
        const int smem = 1024 + p.stages * stage_bytes + (int)sizeof(TcShared) + 64;
        dim3 grid((unsigned)splits, (unsigned)m_chunks, (unsigned)n_tiles);
        wgrad_tc_kernel<<<grid, kThreads, smem, ex.stream>>>(map_a, map_g, p);
        const double bytes = (double)gi.P() * L.cin * 2 + (double)go.P() * L.cout * 2 + (double)p.slice * 4 * (splits > 1 ? splits : 1);
        ex.check("conv_wgrad_tc", bytes, 2.0 * go.P() * L.cout * L.cin * taps);
        if (splits > 1) {
            splitk_sum_kernel<<<(unsigned)((p.slice + 31) / 32), 256, 0, ex.stream>>>(part, p.slice, splits, dW);
            ex.check("splitk_sum", (double)p.slice * 4 * (splits + 1));
        }
    }
    ex.ws.release(m);
    return true;
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
void tc_pack_batch(Exec &ex, const PackJob *jobs_dev, int n_jobs, double bytes) {
    if (ex.dry || n_jobs == 0) return;
    dim3 grid(16, (unsigned)n_jobs);
    pack_weights_batch_kernel<<<grid, 256, 0, ex.stream>>>(jobs_dev);
    ex.check("pack_weights_batch", bytes);
}
