// Convolution forward / data-gradient / weight-gradient as fp32 implicit GEMMs on the CUDA cores.
// This is the strict-precision verification path, and the fallback for shapes the tensor-core
// kernels do not take.  Products and sums are fp32 FMA; operands may be float or bf16.
//
//   fprop: out[p,co]   = sum_{kh,kw,ci} a[p (+) (kh,kw), ci] * W[co,kh,kw,ci]        (Eq. 2, Conv_kxk)
//   dgrad: da[q,ci]    = sum_{kh,kw,co} g[p,co] * W[co,kh,kw,ci],  p*s + (kh,kw) - pad = q
//   wgrad: dW[co,kh,kw,ci] = sum_p g[p,co] * a[p (+) (kh,kw), ci]
#include "common.cuh"

template <class T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16>(const bf16 *p) { return __bfloat162float(*p); }

struct ConvGeom {
    int N, H, W, Ci, Ho, Wo, Co, k, s, pad;
};

// ---- operand loaders: element (m,k) of A and (k,n) of B of the implicit GEMM
template <class TA> struct FpropA {           // m = output pixel, k = (kh,kw,ci)
    const TA *a; ConvGeom g;
    static constexpr bool k_fast = true;
    __device__ float operator()(int m, int kk) const {
        int wo = m % g.Wo, t = m / g.Wo, ho = t % g.Ho, n = t / g.Ho;
        int ci = kk % g.Ci, tap = kk / g.Ci, kw = tap % g.k, kh = tap / g.k;
        int y = ho * g.s + kh - g.pad, x = wo * g.s + kw - g.pad;
        if (y < 0 || y >= g.H || x < 0 || x >= g.W) return 0.f;
        return ldf(a + (((size_t)n * g.H + y) * g.W + x) * g.Ci + ci);
    }
};
__device__ __forceinline__ float round_w(float w, bool to_bf16) { return to_bf16 ? __bfloat162float(__float2bfloat16_rn(w)) : w; }
struct FpropB {                               // k = (kh,kw,ci), n = co ; W[co][kh][kw][ci]
    const float *w; int K; bool wb;           // wb: weights take part as bf16 values (mode 0)
    static constexpr bool k_fast = true;
    __device__ float operator()(int kk, int n) const { return round_w(w[(size_t)n * K + kk], wb); }
};
template <class TG> struct DgradA {           // m = input pixel, k = (kh,kw,co)
    const TG *gq; ConvGeom g;
    static constexpr bool k_fast = true;
    __device__ float operator()(int m, int kk) const {
        int x = m % g.W, t = m / g.W, y = t % g.H, n = t / g.H;
        int co = kk % g.Co, tap = kk / g.Co, kw = tap % g.k, kh = tap / g.k;
        int yy = y + g.pad - kh, xx = x + g.pad - kw;
        if (yy < 0 || xx < 0 || yy % g.s || xx % g.s) return 0.f;
        int ho = yy / g.s, wo = xx / g.s;
        if (ho >= g.Ho || wo >= g.Wo) return 0.f;
        return ldf(gq + (((size_t)n * g.Ho + ho) * g.Wo + wo) * g.Co + co);
    }
};
struct DgradB {                               // k = (kh,kw,co), n = ci
    const float *w; ConvGeom g; bool wb;
    static constexpr bool k_fast = false;
    __device__ float operator()(int kk, int n) const {
        int co = kk % g.Co, tap = kk / g.Co;
        return round_w(w[((size_t)co * g.k * g.k + tap) * g.Ci + n], wb);
    }
};
template <class TG> struct WgradA {           // m = co, k = output pixel
    const TG *gq; ConvGeom g;
    static constexpr bool k_fast = false;
    __device__ float operator()(int m, int kk) const { return ldf(gq + (size_t)kk * g.Co + m); }
};
template <class TA> struct WgradB {           // k = output pixel, n = (kh,kw,ci)
    const TA *a; ConvGeom g;
    static constexpr bool k_fast = false;
    __device__ float operator()(int kk, int n) const {
        int wo = kk % g.Wo, t = kk / g.Wo, ho = t % g.Ho, b = t / g.Ho;
        int ci = n % g.Ci, tap = n / g.Ci, kw = tap % g.k, kh = tap / g.k;
        int y = ho * g.s + kh - g.pad, x = wo * g.s + kw - g.pad;
        if (y < 0 || y >= g.H || x < 0 || x >= g.W) return 0.f;
        return ldf(a + (((size_t)b * g.H + y) * g.W + x) * g.Ci + ci);
    }
};

// ---- epilogues
struct EpiCouple {                            // out = partner + sign*acc (sign 0: plain store); out/partner may be split pairs
    Pair out, partner; int sign;
    __device__ void operator()(int m, int n, float v, int) const { out.couple(m, n, v, partner, sign); }
};
struct EpiPlain {                             // row-major [M][N] (+ split-K slice)
    float *out; int N; size_t slice;
    __device__ void operator()(int m, int n, float v, int z) const { out[z * slice + (size_t)m * N + n] = v; }
};

template <int BN, class AL, class BL, class EP>
__global__ __launch_bounds__(256) void gemm_simt_kernel(AL al, BL bl, EP ep, int M, int N, int K, int k_per_split) {
    pdl_enter();
    constexpr int BM = 64, BK = 16, TN = BN / 16;
    __shared__ float As[BK][BM + 1];
    __shared__ float Bs[BK][BN + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int kbeg = blockIdx.z * k_per_split;
    int kend = kbeg + k_per_split; if (kend > K) kend = K;
    float acc[4][TN];
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < TN; j++) acc[i][j] = 0.f;

    for (int k0 = kbeg; k0 < kend; k0 += BK) {
#pragma unroll
        for (int i = 0; i < (BM * BK) / 256; i++) {
            int e = tid + i * 256, mm, kk;
            if (AL::k_fast) { kk = e % BK; mm = e / BK; } else { mm = e % BM; kk = e / BM; }
            As[kk][mm] = (m0 + mm < M && k0 + kk < kend) ? al(m0 + mm, k0 + kk) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < (BN * BK + 255) / 256; i++) {
            int e = tid + i * 256, nn, kk;
            if (BL::k_fast) { kk = e % BK; nn = e / BK; } else { nn = e % BN; kk = e / BN; }
            if (e < BN * BK) Bs[kk][nn] = (n0 + nn < N && k0 + kk < kend) ? bl(k0 + kk, n0 + nn) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; kk++) {
            float a[4], b[TN];
#pragma unroll
            for (int i = 0; i < 4; i++) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < TN; j++) b[j] = Bs[kk][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; i++)
#pragma unroll
                for (int j = 0; j < TN; j++) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < TN; j++) {
            int m = m0 + ty * 4 + i, n = n0 + tx + 16 * j;
            if (m < M && n < N) ep(m, n, acc[i][j], blockIdx.z);
        }
}

template <class AL, class BL, class EP>
static void launch_gemm(Exec &ex, const char *what, AL al, BL bl, EP ep, int M, int N, int K, int splits, int k_per_split,
                        double bytes) {
    if (N <= 16) {
        dim3 grid((M + 63) / 64, (N + 15) / 16, splits);
        launch(ex, gemm_simt_kernel<16, AL, BL, EP>, grid, 256, 0, al, bl, ep, M, N, K, k_per_split);
    } else if (N <= 32) {
        dim3 grid((M + 63) / 64, (N + 31) / 32, splits);
        launch(ex, gemm_simt_kernel<32, AL, BL, EP>, grid, 256, 0, al, bl, ep, M, N, K, k_per_split);
    } else {
        dim3 grid((M + 63) / 64, (N + 63) / 64, splits);
        launch(ex, gemm_simt_kernel<64, AL, BL, EP>, grid, 256, 0, al, bl, ep, M, N, K, k_per_split);
    }
    ex.check(what, bytes, 2.0 * M * N * (double)K);
}

static ConvGeom geom_of(Geom gi, const Layer &L) {
    ConvGeom g;
    g.N = gi.N; g.H = gi.H; g.W = gi.W; g.Ci = L.cin; g.Co = L.cout; g.k = L.k; g.s = L.stride; g.pad = L.k / 2;
    g.Ho = conv_out(gi.H, L.k, L.stride); g.Wo = conv_out(gi.W, L.k, L.stride);
    return g;
}

void conv_fprop_simt(Exec &ex, const void *a, bool a_bf16, Geom gi, const Layer &L, Pair out, Pair partner, int sign) {
    ConvGeom g = geom_of(gi, L);
    const int M = g.N * g.Ho * g.Wo, N = g.Co, K = g.k * g.k * g.Ci;
    ex.flops += 2ull * M * N * K;
    if (ex.dry) return;
    EpiCouple ep{out, partner, sign};
    FpropB bl{L.W, K, a_bf16};
    const double bytes = (double)g.N * g.H * g.W * g.Ci * (a_bf16 ? 2 : 4) + (double)M * N * (sign ? 8 : 4) + (double)N * K * 4;
    if (a_bf16) launch_gemm(ex, "conv_fprop_simt", FpropA<bf16>{(const bf16 *)a, g}, bl, ep, M, N, K, 1, K, bytes);
    else launch_gemm(ex, "conv_fprop_simt", FpropA<float>{(const float *)a, g}, bl, ep, M, N, K, 1, K, bytes);
}

void conv_dgrad_simt(Exec &ex, const void *gq, bool g_bf16, Geom gi, const Layer &L, float *da) {
    ConvGeom g = geom_of(gi, L);
    const int M = g.N * g.H * g.W, N = g.Ci, K = g.k * g.k * g.Co;
    ex.flops += 2ull * g.N * g.Ho * g.Wo * N * K;
    if (ex.dry) return;
    EpiPlain ep{da, N, 0};
    DgradB bl{L.W, g, g_bf16};
    const double bytes = (double)g.N * g.Ho * g.Wo * g.Co * (g_bf16 ? 2 : 4) + (double)M * N * 4 + (double)N * K * 4;
    if (g_bf16) launch_gemm(ex, "conv_dgrad_simt", DgradA<bf16>{(const bf16 *)gq, g}, bl, ep, M, N, K, 1, K, bytes);
    else launch_gemm(ex, "conv_dgrad_simt", DgradA<float>{(const float *)gq, g}, bl, ep, M, N, K, 1, K, bytes);
}

// fixed-order sum of split-K slices
__global__ void splitk_reduce_kernel(const float *__restrict__ part, size_t n, int splits, float *__restrict__ out) {
    pdl_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int z = 0; z < splits; z++) s += part[(size_t)z * n + i];
        out[i] = s;
    }
}

void conv_wgrad_simt(Exec &ex, const void *gq, bool g_bf16, const void *a, bool a_bf16, Geom gi, const Layer &L, float *dW) {
    ConvGeom g = geom_of(gi, L);
    const int M = g.Co, N = g.k * g.k * g.Ci, K = g.N * g.Ho * g.Wo;
    ex.flops += 2ull * M * N * (size_t)K;
    // split the pixel sum so that the grid fills the machine; slices are summed in fixed order
    int tiles = ((M + 63) / 64) * ((N + 63) / 64);
    int splits = (ex.ctx->sm_count * 2 + tiles - 1) / tiles;
    int max_splits = (K + 255) / 256; if (splits > max_splits) splits = max_splits; if (splits < 1) splits = 1;
    int kps = (((K + splits - 1) / splits) + 15) / 16 * 16;
    splits = (K + kps - 1) / kps;
    size_t m = ex.ws.mark();
    float *part = splits > 1 ? ex.ws.get<float>((size_t)splits * M * N) : dW;
    if (!ex.dry) {
        EpiPlain ep{part, N, (size_t)M * N};
        const double bytes = (double)K * g.Co * (g_bf16 ? 2 : 4) + (double)g.N * g.H * g.W * g.Ci * (a_bf16 ? 2 : 4) + (double)M * N * 4;
#define RV_WG(TG, TA) launch_gemm(ex, "conv_wgrad_simt", WgradA<TG>{(const TG *)gq, g}, WgradB<TA>{(const TA *)a, g}, ep, M, N, K, splits, kps, bytes)
        if (g_bf16 && a_bf16) RV_WG(bf16, bf16);
        else if (g_bf16) RV_WG(bf16, float);
        else if (a_bf16) RV_WG(float, bf16);
        else RV_WG(float, float);
#undef RV_WG
        if (splits > 1) {
            size_t n = (size_t)M * N;
            int grid = (int)((n + 255) / 256); if (grid > ex.ctx->sm_count * 8) grid = ex.ctx->sm_count * 8;
            launch(ex, splitk_reduce_kernel, grid, 256, 0, part, n, splits, dW);
            ex.check("splitk_reduce");
        }
    }
    ex.ws.release(m);
}
