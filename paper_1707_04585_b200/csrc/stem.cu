// The stem: a bare convolution of the 3-channel image (3x3 stride 1, or 7x7 stride 2), fp32 in both
// precision modes, forward and weight gradient.  With so few input channels the contraction per
// output pixel is short (K = k*k*3 = 27 or 147) and a tensor-core tile would be mostly padding, so
// these are register-tiled CUDA-core kernels: the image patches of a tile of output pixels (128
// forward, 64 for the weight gradient) are gathered into shared memory once and every thread keeps a
// small block of the result in registers.
//
//   fprop: out[p, co]      = sum_{kh,kw,ci} img[p*s + (kh,kw) - pad, ci] * W[co, kh, kw, ci]
//   wgrad: dW[co, kh,kw,ci] = sum_p g[p, co] * img[p*s + (kh,kw) - pad, ci]
// (the stem has no data gradient: nothing lies below the image).
#include "common.cuh"

namespace {

constexpr int kPx = 64;            // output pixels per chunk of the weight gradient
constexpr int kFPx = 128;          // output pixels per tile of the forward kernel

struct StemGeom { int N, H, W, Ci, Ho, Wo, Co, k, s, pad, K; };

// patch element kk = (kh, kw, ci) of the output pixel whose window starts at (y0, x0) of image n; zero outside
// the image.  Without branches (the load of an outside element reads the image's first pixel and is dropped),
// so that the loads of an unrolled gather loop are in flight together.
__device__ __forceinline__ float patch_at(const float *__restrict__ img, const StemGeom &g, size_t nbase, int y0, int x0, int koff, bool live) {
    const int kh = koff >> 16, kw = (koff >> 8) & 0xff, ci = koff & 0xff;
    const int y = y0 + kh, x = x0 + kw;
    const bool in = live && (unsigned)y < (unsigned)g.H && (unsigned)x < (unsigned)g.W;
    const size_t idx = in ? nbase + ((size_t)y * g.W + x) * g.Ci + ci : 0;
    const float v = __ldg(img + idx);
    return in ? v : 0.f;
}

__device__ __forceinline__ void fill_koff(const StemGeom &g, int *koff, int tid, int nthreads) {
    for (int kk = tid; kk < g.K; kk += nthreads) {
        const int ci = kk % g.Ci, tap = kk / g.Ci, kw = tap % g.k, kh = tap / g.k;
        koff[kk] = (kh << 16) | (kw << 8) | ci;
    }
}

// 256 threads, tiles of 128 output pixels: thread (tx = tid & 7, ty = tid >> 3) owns pixels ty*4 .. ty*4+3 of the tile and, per pass,
// output channels co0 + tx*CO_T .. + CO_T-1.  Shared memory: the weights transposed to [K][cop]
// (cop = Co rounded up to 8*CO_T), the tile's patches [K][128], the tap table.
template <int CO_T>
__global__ void __launch_bounds__(256) stem_fprop_kernel(const float *__restrict__ img, const float *__restrict__ W, Pair out,
                                                         StemGeom g, int cop, int n_tiles) {
    extern __shared__ float sm[];
    float *Ws = sm;                               // [K][cop]
    float *As = Ws + (size_t)g.K * cop;           // [K][kFPx]
    int *koff = reinterpret_cast<int *>(As + (size_t)g.K * kFPx);
    const int tid = threadIdx.x, tx = tid & 7, ty = tid >> 3;
    fill_koff(g, koff, tid, 256);
    for (int e = tid; e < g.K * cop; e += 256) {
        const int co = e % cop, kk = e / cop;
        Ws[e] = co < g.Co ? W[(size_t)co * g.K + kk] : 0.f;
    }
    pdl_enter();
    const int P = g.N * g.Ho * g.Wo;
    const int px = tid & (kFPx - 1), kk0 = tid >> 7;      // this thread gathers pixel px, patch elements kk0, kk0 + 2, ...
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        __syncthreads();                                   // tables ready / the previous tile's patches consumed
        {
            const int p = t * kFPx + px;
            const bool live = p < P;
            const int wo = p % g.Wo, r = p / g.Wo, ho = r % g.Ho, n = r / g.Ho;
            const size_t nbase = (size_t)n * g.H * g.W * g.Ci;
            const int y0 = ho * g.s - g.pad, x0 = wo * g.s - g.pad;
#pragma unroll 8
            for (int kk = kk0; kk < g.K; kk += 2) As[kk * kFPx + px] = patch_at(img, g, nbase, y0, x0, koff[kk], live);
        }
        __syncthreads();
        for (int co0 = 0; co0 < cop; co0 += 8 * CO_T) {
            float acc[4][CO_T];
#pragma unroll
            for (int i = 0; i < 4; i++)
#pragma unroll
                for (int j = 0; j < CO_T; j++) acc[i][j] = 0.f;
            const float *wrow = Ws + co0 + tx * CO_T;
#pragma unroll 3
            for (int kk = 0; kk < g.K; kk++) {
                const float4 a = *reinterpret_cast<const float4 *>(As + kk * kFPx + ty * 4);
                float w[CO_T];
#pragma unroll
                for (int j = 0; j < CO_T; j += 4) {
                    const float4 v = *reinterpret_cast<const float4 *>(wrow + (size_t)kk * cop + j);
                    w[j] = v.x; w[j + 1] = v.y; w[j + 2] = v.z; w[j + 3] = v.w;
                }
#pragma unroll
                for (int j = 0; j < CO_T; j++) {
                    acc[0][j] = fmaf(a.x, w[j], acc[0][j]); acc[1][j] = fmaf(a.y, w[j], acc[1][j]);
                    acc[2][j] = fmaf(a.z, w[j], acc[2][j]); acc[3][j] = fmaf(a.w, w[j], acc[3][j]);
                }
            }
            const int co = co0 + tx * CO_T;
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const int p = t * kFPx + ty * 4 + i;
                if (p >= P) continue;
#pragma unroll
                for (int j = 0; j < CO_T; j += 4)
                    if (co + j < g.Co) out.store4((size_t)p, co + j, make_float4(acc[i][j], acc[i][j + 1], acc[i][j + 2], acc[i][j + 3]));
            }
        }
    }
}

// 256 threads = G groups x S pixel lanes.  Group (cg, kg) owns the CO_T x KK_T block of dW at output channels
// cg*CO_T.., patch elements kg*KK_T..; lane `sub` of the group adds the pixels sub, sub + S, ... of every
// 64-pixel chunk the CTA walks.  At the end the lanes are added in order through shared memory and the CTA
// writes one partial [Co][K]; splitk_reduce adds the partials in order.
template <int CO_T, int KK_T>
__global__ void __launch_bounds__(256) stem_wgrad_kernel(const float *__restrict__ img, const float *__restrict__ gout, float *__restrict__ part,
                                                         StemGeom g, int cop, int kp, int n_cg, int G, int S, int n_chunks) {
    extern __shared__ float sm[];
    float *Gs = sm;                               // [kPx][cop]
    float *As = Gs + (size_t)kPx * cop;           // [kPx][kp]
    int *koff = reinterpret_cast<int *>(As + (size_t)kPx * kp);
    const int tid = threadIdx.x;
    fill_koff(g, koff, tid, 256);
    pdl_enter();
    const int grp = tid % G, sub = tid / G;
    const bool worker = sub < S;
    const int cg = grp % n_cg, kg = grp / n_cg;
    float acc[CO_T][KK_T];
#pragma unroll
    for (int i = 0; i < CO_T; i++)
#pragma unroll
        for (int j = 0; j < KK_T; j++) acc[i][j] = 0.f;
    const int P = g.N * g.Ho * g.Wo;
    const int px = tid & (kPx - 1), kk0 = tid >> 6;      // gathers pixel px, patch elements kk0, kk0 + 4, ...
    for (int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        __syncthreads();
        {
            const int p = c * kPx + px;
            const bool live = p < P;
            const int wo = p % g.Wo, r = p / g.Wo, ho = r % g.Ho, n = r / g.Ho;
            const size_t nbase = (size_t)n * g.H * g.W * g.Ci;
            const int y0 = ho * g.s - g.pad, x0 = wo * g.s - g.pad;
#pragma unroll 8
            for (int kk = kk0; kk < kp; kk += 4) As[px * kp + kk] = patch_at(img, g, nbase, y0, x0, koff[kk < g.K ? kk : 0], live && kk < g.K);
        }
        for (int e = tid; e < kPx * cop; e += 256) {
            const int co = e % cop, q = e / cop;
            const int p = c * kPx + q;
            Gs[e] = (p < P && co < g.Co) ? gout[(size_t)p * g.Co + co] : 0.f;
        }
        __syncthreads();
        if (worker) {
            for (int q = sub; q < kPx; q += S) {
                float gv[CO_T], av[KK_T];
#pragma unroll
                for (int i = 0; i < CO_T; i += 4) {
                    const float4 v = *reinterpret_cast<const float4 *>(Gs + q * cop + cg * CO_T + i);
                    gv[i] = v.x; gv[i + 1] = v.y; gv[i + 2] = v.z; gv[i + 3] = v.w;
                }
#pragma unroll
                for (int j = 0; j < KK_T; j += 4) {
                    const float4 v = *reinterpret_cast<const float4 *>(As + q * kp + kg * KK_T + j);
                    av[j] = v.x; av[j + 1] = v.y; av[j + 2] = v.z; av[j + 3] = v.w;
                }
#pragma unroll
                for (int i = 0; i < CO_T; i++)
#pragma unroll
                    for (int j = 0; j < KK_T; j++) acc[i][j] = fmaf(gv[i], av[j], acc[i][j]);
            }
        }
    }
    // lanes of a group are added in order, one block element at a time through shared memory
    __syncthreads();
    float *red = sm;                              // [S][G] floats (S*G <= 256)
    float *mine = part + (size_t)blockIdx.x * g.Co * g.K;
#pragma unroll
    for (int i = 0; i < CO_T; i++)
#pragma unroll
        for (int j = 0; j < KK_T; j++) {
            if (worker) red[sub * G + grp] = acc[i][j];
            __syncthreads();
            if (worker && sub == 0) {
                float s = red[grp];
                for (int y = 1; y < S; y++) s += red[y * G + grp];
                const int co = cg * CO_T + i, kk = kg * KK_T + j;
                if (co < g.Co && kk < g.K) mine[(size_t)co * g.K + kk] = s;
            }
            __syncthreads();
        }
}

// dW[i] = sum of the per-CTA partials, one warp per element: lane l adds the partials l, l + 32, ... and the
// lanes are combined by a shuffle tree, so the order of additions is fixed by `parts` alone
__global__ void stem_sum_kernel(const float *__restrict__ part, size_t n, int parts, float *__restrict__ out) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = ((size_t)gridDim.x * blockDim.x) >> 5;
    for (size_t i = warp; i < n; i += n_warps) {
        float s = 0.f;
        for (int z = lane; z < parts; z += 32) s += part[(size_t)z * n + i];
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) out[i] = s;
    }
}

StemGeom stem_geom(Geom gi, const Layer &L) {
    StemGeom g;
    g.N = gi.N; g.H = gi.H; g.W = gi.W; g.Ci = L.cin; g.Co = L.cout; g.k = L.k; g.s = L.stride; g.pad = L.k / 2;
    g.Ho = conv_out(gi.H, L.k, L.stride); g.Wo = conv_out(gi.W, L.k, L.stride);
    g.K = L.k * L.k * L.cin;
    return g;
}
int round_up(int x, int m) { return (x + m - 1) / m * m; }

}  // namespace

// image: fp32 [N,H,W,cin]; out: the stem's output (a plain tensor or the halves of stage 0's pair, float or fixed point)
bool stem_fprop(Exec &ex, const float *img, Geom gi, const Layer &L, Pair out) {
    const StemGeom g = stem_geom(gi, L);
    if (L.cin > 255 || L.k > 255 || L.cout % 4 || (out.c1 && out.c0 % 4)) return false;
    const int CO_T = L.cout >= 64 ? 8 : 4;
    const int cop = round_up(L.cout, 8 * CO_T);
    const size_t smem = ((size_t)g.K * cop + (size_t)g.K * kFPx) * 4 + (size_t)g.K * 4;
    if (smem > 200 * 1024) return false;
    ex.flops += 2ull * g.N * g.Ho * g.Wo * g.Co * g.K;
    if (ex.dry) return true;
    const int P = g.N * g.Ho * g.Wo, n_tiles = (P + kFPx - 1) / kFPx;
    int per_sm = (int)((220 * 1024) / (smem + 1024)); if (per_sm > 8) per_sm = 8; if (per_sm < 1) per_sm = 1;
    int grid = ex.ctx->sm_count * per_sm; if (grid > n_tiles) grid = n_tiles;
    static OncePerDevice once;
    if (once.first(ex.ctx->device)) {
        cudaFuncSetAttribute(stem_fprop_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        cudaFuncSetAttribute(stem_fprop_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    }
    if (CO_T == 8) launch(ex, stem_fprop_kernel<8>, grid, 256, smem, img, L.W, out, g, cop, n_tiles);
    else launch(ex, stem_fprop_kernel<4>, grid, 256, smem, img, L.W, out, g, cop, n_tiles);
    ex.check("stem_fprop", (double)g.N * g.H * g.W * g.Ci * 4 + (double)P * g.Co * 4 + (double)g.Co * g.K * 4, 2.0 * P * g.Co * g.K);
    return true;
}

// gout: fp32 [P, cout] gradient w.r.t. the stem output; dW: [cout][k][k][cin]
bool stem_wgrad(Exec &ex, const float *img, const float *gout, Geom gi, const Layer &L, float *dW) {
    const StemGeom g = stem_geom(gi, L);
    if (L.cin > 255 || L.k > 255) return false;
    const bool big = L.cout >= 64;
    const int CO_T = big ? 8 : 4, KK_T = big ? 12 : 4;
    const int cop = round_up(L.cout, CO_T), kp = round_up(g.K, KK_T);
    const int n_cg = cop / CO_T, n_kg = kp / KK_T, G = n_cg * n_kg;
    if (G > 256) return false;
    const int S = 256 / G;
    const size_t smem = ((size_t)kPx * cop + (size_t)kPx * kp) * 4 + (size_t)g.K * 4;
    if (smem > 200 * 1024) return false;
    const int P = g.N * g.Ho * g.Wo, n_chunks = (P + kPx - 1) / kPx;
    int grid = ex.ctx->sm_count * 2; if (grid > n_chunks) grid = n_chunks;
    ex.flops += 2ull * P * g.Co * g.K;
    size_t m = ex.ws.mark();
    float *part = ex.ws.get<float>((size_t)grid * g.Co * g.K);
    if (!ex.dry) {
        static OncePerDevice once;
        if (once.first(ex.ctx->device)) {
            cudaFuncSetAttribute(stem_wgrad_kernel<8, 12>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            cudaFuncSetAttribute(stem_wgrad_kernel<4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        }
        if (big) launch(ex, stem_wgrad_kernel<8, 12>, grid, 256, smem, img, gout, part, g, cop, kp, n_cg, G, S, n_chunks);
        else launch(ex, stem_wgrad_kernel<4, 4>, grid, 256, smem, img, gout, part, g, cop, kp, n_cg, G, S, n_chunks);
        ex.check("stem_wgrad", (double)g.N * g.H * g.W * g.Ci * 4 + (double)P * g.Co * 4, 2.0 * P * g.Co * g.K);
        const size_t n = (size_t)g.Co * g.K;
        int sg = (int)((n + 7) / 8); if (sg > ex.ctx->sm_count * 8) sg = ex.ctx->sm_count * 8;      // eight warps per block
        launch(ex, stem_sum_kernel, sg, 256, 0, (const float *)part, n, grid, dW);
        ex.check("stem_sum", (double)n * 4 * (grid + 1));
    }
    ex.ws.release(m);
    return true;
}
