// HBM-bound kernels: BN batch statistics, BN+ReLU apply and backward, concat/cast, max-pool,
// classification head, SGD.  All reductions are two-stage with a fixed summation order, so a
// residual function recomputed in the backward pass reproduces the forward bit for bit.
#include "common.cuh"
#include "conv_epilogue.cuh"
#include <math.h>

cudaEvent_t revnet_ctx::next_event() {
    if (ev_used == ev_pool.size()) {
        cudaEvent_t e;
        cudaEventCreate(&e);
        ev_pool.push_back(e);
    }
    return ev_pool[ev_used++];
}

unsigned long long *Exec::stamp_slot() {
    if (dry || !ctx->stamping || !ctx->stamps || ctx->stamp_next >= kStampSlots) return nullptr;
    pending_slot = ctx->stamp_next++;
    return ctx->stamps + pending_slot;
}

void Exec::check(const char *what, double bytes, double flops) {
    launches++;
    if (pending_slot >= 0) { ctx->stamp_recs.push_back(StampRec{what, bytes, flops, pending_slot}); pending_slot = -1; }
    cudaError_t e = cudaPeekAtLastError();
    if (e != cudaSuccess && !failed) {
        failed = true;
        ctx->err = std::string(what) + ": " + cudaGetErrorString(e);
    }
    if (ctx->profiling) {
        cudaEvent_t ev = ctx->next_event();
        cudaEventRecord(ev, stream);
        ctx->prof.push_back(ProfRec{what, bytes, flops, ev});
    }
}
// Keeps the stream busy for `ns` nanoseconds (bounded) so that the host gets ahead of the device:
// the per-kernel events of a profiled step then measure kernels that were already queued, not the
// host's launch rate.
__global__ void profile_hold_kernel(unsigned long long ns) {
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (int i = 0; i < 100000; i++) {
        __nanosleep(1000);
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        if (t - t0 >= ns) break;
    }
}
void Exec::mark(const char *what) {
    if (ctx->profiling && !dry && hold_ns) {
        profile_hold_kernel<<<1, 1, 0, stream>>>(hold_ns);
        hold_ns = 0;
    }
    if (ctx->profiling && !dry) {
        cudaEvent_t ev = ctx->next_event();
        cudaEventRecord(ev, stream);
        ctx->prof.push_back(ProfRec{what, 0, 0, ev});
    }
}

static inline int cdiv(size_t a, size_t b) { return (int)((a + b - 1) / b); }

__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void st4(bf16 *p, float4 v) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&lo);
    u.y = *reinterpret_cast<uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(p) = u;
}

// ------------------------------------------------------------------ column reductions
// Shape of the launch used by every per-channel reduction over a [P,C] tensor: a CTA owns a slab
// of SW channel quads and a range of rows; threadIdx.y strides the rows.
struct RedShape { int SW, RPP, slabs, chunks, rows_per_cta; };
static RedShape red_shape(size_t P, int C, int sm) {
    RedShape r;
    int C4 = C / 4;
    r.SW = C4 < 128 ? C4 : 128;
    r.RPP = 256 / r.SW; if (r.RPP < 1) r.RPP = 1;
    r.slabs = cdiv(C4, r.SW);
    size_t want = (size_t)sm * 4 / r.slabs; if (want < 1) want = 1;
    size_t rows = (P + want - 1) / want;
    size_t min_rows = (size_t)r.RPP * 8;
    if (rows < min_rows) rows = min_rows;
    r.rows_per_cta = (int)rows;
    r.chunks = cdiv(P, rows);
    return r;
}

// part layout: [chunk][2][C]
template <int MODE>   // 0: sum t, sum t^2 ; 1: sum db, sum db*xhat (BN+ReLU backward)
__global__ void col_reduce_kernel(Pair t, const float *__restrict__ da, size_t P, int rows_per_cta, BnRef bn,
                                  float *__restrict__ part) {
    pdl_enter();
    extern __shared__ float4 sm4[];
    const int C = t.C(), C4 = C / 4, SW = blockDim.x, RPP = blockDim.y;
    const int q = blockIdx.y * SW + threadIdx.x;
    const bool valid = q < C4;
    const size_t r0 = (size_t)blockIdx.x * rows_per_cta;
    size_t r1 = r0 + rows_per_cta; if (r1 > P) r1 = P;
    float4 s = make_float4(0, 0, 0, 0), ss = s;
    if (valid) {
        float4 sc, sh, mu, rs;
        if (MODE == 1) bn_coef4(bn, q * 4, sc, sh, mu, rs);
        for (size_t r = r0 + threadIdx.y; r < r1; r += RPP) {
            float4 v = t.ld4(r, q * 4);
            if (MODE == 0) {
                s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
                ss.x += v.x * v.x; ss.y += v.y * v.y; ss.z += v.z * v.z; ss.w += v.w * v.w;
            } else {
                float4 g = ld4(da + r * C + q * 4);
                float dx = fmaf(sc.x, v.x, sh.x) > 0.f ? g.x : 0.f, dy = fmaf(sc.y, v.y, sh.y) > 0.f ? g.y : 0.f;
                float dz = fmaf(sc.z, v.z, sh.z) > 0.f ? g.z : 0.f, dw = fmaf(sc.w, v.w, sh.w) > 0.f ? g.w : 0.f;
                s.x += dx; s.y += dy; s.z += dz; s.w += dw;
                ss.x += dx * ((v.x - mu.x) * rs.x); ss.y += dy * ((v.y - mu.y) * rs.y);
                ss.z += dz * ((v.z - mu.z) * rs.z); ss.w += dw * ((v.w - mu.w) * rs.w);
            }
        }
    }
    sm4[(threadIdx.y * SW + threadIdx.x) * 2 + 0] = s;
    sm4[(threadIdx.y * SW + threadIdx.x) * 2 + 1] = ss;
    __syncthreads();
    if (threadIdx.y == 0 && valid) {
        for (int y = 1; y < RPP; y++) {
            float4 a = sm4[(y * SW + threadIdx.x) * 2], b = sm4[(y * SW + threadIdx.x) * 2 + 1];
            s.x += a.x; s.y += a.y; s.z += a.z; s.w += a.w;
            ss.x += b.x; ss.y += b.y; ss.z += b.z; ss.w += b.w;
        }
        st4(part + ((size_t)blockIdx.x * 2 + 0) * C + q * 4, s);
        st4(part + ((size_t)blockIdx.x * 2 + 1) * C + q * 4, ss);
    }
}

// one warp per channel: lanes stride the per-CTA partials, double accumulation, fixed butterfly order
__device__ __forceinline__ void warp_sum2(const float *__restrict__ part, int chunks, int C, int c, double &s, double &ss) {
    const int lane = threadIdx.x & 31;
    s = 0; ss = 0;
    for (int i = lane; i < chunks; i += 32) { s += part[((size_t)i * 2) * C + c]; ss += part[((size_t)i * 2 + 1) * C + c]; }
    for (int o = 16; o; o >>= 1) { s += __shfl_xor_sync(0xffffffffu, s, o); ss += __shfl_xor_sync(0xffffffffu, ss, o); }
}

__global__ void bn_stats_finalize(const float *__restrict__ part, int chunks, int C, double invP, float eps,
                                  float *mean, float *rstd) {
    pdl_enter();
    const int c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (c >= C) return;
    double s, ss;
    warp_sum2(part, chunks, C, c, s, ss);
    if ((threadIdx.x & 31) == 0) {
        double mu = s * invP, var = ss * invP - mu * mu;
        if (var < 0) var = 0;
        mean[c] = (float)mu; rstd[c] = (float)(1.0 / sqrt(var + (double)eps));
    }
}

// coef: [3][C] = gamma*rstd, gamma*rstd*dbeta/M, gamma*rstd*dgamma/M
__global__ void bn_bwd_finalize(const float *__restrict__ part, int chunks, int C, double invP,
                                const float *__restrict__ gamma, const float *__restrict__ rstd,
                                float *dgamma, float *dbeta, float *coef) {
    pdl_enter();
    const int c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (c >= C) return;
    double s, ss;
    warp_sum2(part, chunks, C, c, s, ss);
    if ((threadIdx.x & 31) == 0) {
        dbeta[c] = (float)s; dgamma[c] = (float)ss;
        double gr = (double)gamma[c] * (double)rstd[c];
        coef[c] = (float)gr; coef[C + c] = (float)(gr * s * invP); coef[2 * C + c] = (float)(gr * ss * invP);
    }
}

Moments mom_alloc(Exec &ex, int C, bool with_part) {
    Moments m;
    float *p = ex.ws.get<float>((size_t)2 * C);
    m.mean = p; m.rstd = p + C;
    if (with_part) {
        // a fused convolution runs at most two CTAs per SM, one record of 2C floats each
        m.part_cap = (size_t)2 * ex.ctx->sm_count * 2 * C;
        m.part = ex.ws.get<float>(m.part_cap);
    }
    return m;
}

__global__ void __launch_bounds__(256) moments_finalize_kernel(const float *part, int parts, int C, double inv_count, float eps,
                                                             float *mean, float *rstd) {
    pdl_enter();
    __shared__ double red[256 * 4], tot[128 * 4];
    const int R = C >> 1, tid = threadIdx.x;
    for (int slot0 = 0; slot0 < R; slot0 += 128) {
        const int cw = R - slot0 < 128 ? R - slot0 : 128;
        tc::reduce_records<256>(part, parts, C, slot0, cw, red, tot, tid);
        for (int lc = tid; lc < cw * 2; lc += 256) {
            const int k = lc >> 2, j = lc & 3, ch = (slot0 >> 1) * 4 + lc;
            tc::moments_of(tot[(2 * k) * 4 + j], tot[(2 * k + 1) * 4 + j], inv_count, eps, mean[ch], rstd[ch]);
        }
        tc::named_barrier(1, 256);
    }
}

void mom_finalize(Exec &ex, Moments &m, int C) {
    if (!m.pending) return;
    if (!ex.dry) {
        launch(ex, moments_finalize_kernel, 1, 256, 0, (const float *)m.part, m.parts, C, m.inv_count, ex.eps, m.mean, m.rstd);
        ex.check("bn_stats_finalize");
    }
    m.pending = false;
}

void bn_stats(Exec &ex, Pair t, size_t P, Moments mo) {
    const int C = t.C();
    RedShape r = red_shape(P, C, ex.ctx->sm_count);
    size_t m = ex.ws.mark();
    float *part = ex.ws.get<float>((size_t)r.chunks * 2 * C);
    if (!ex.dry) {
        dim3 grid(r.chunks, r.slabs), block(r.SW, r.RPP);
        launch(ex, col_reduce_kernel<0>, grid, block, (size_t)r.SW * r.RPP * 32, t, nullptr, P, r.rows_per_cta, BnRef{}, part);
        ex.check("bn_stats_partial", (double)P * C * 4);
        launch(ex, bn_stats_finalize, cdiv((size_t)C * 32, 128), 128, 0, part, r.chunks, C, 1.0 / (double)P, ex.eps, mo.mean, mo.rstd);
        ex.check("bn_stats_finalize");
    }
    ex.ws.release(m);
}

// A thread keeps one channel quad (scale and shift stay in registers) and strides the rows, four rows in flight;
// row_step = threads of the grid / C4 (the launch makes that a whole number): no division per element.
template <class TO>
__global__ void __launch_bounds__(256) bn_relu_apply_kernel(Pair t, size_t P, int C4, BnRef bn, TO *__restrict__ a, unsigned long long *stamp) {
    pdl_enter();
    stamp_begin(stamp);
    const int C = C4 * 4;
    const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, nth = (size_t)gridDim.x * blockDim.x;
    const int q = (int)(gtid % C4), c = q * 4;
    const size_t row0 = gtid / C4, row_step = nth / C4;
    float4 sc, sh, mu, rs;
    bn_coef4(bn, c, sc, sh, mu, rs);
    for (size_t rb = row0; rb < P; rb += 4 * row_step) {
        // all four loads leave before anything waits on one: rows beyond the end read the last row again and are not stored
        float4 v[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const size_t row = rb + j * row_step;
            v[j] = t.ld4_raw(row < P ? row : P - 1, c);
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const size_t row = rb + j * row_step;
            if (row >= P) continue;
            v[j] = t.from_raw(v[j]);
            float4 o;
            o.x = fmaxf(fmaf(sc.x, v[j].x, sh.x), 0.f); o.y = fmaxf(fmaf(sc.y, v[j].y, sh.y), 0.f);
            o.z = fmaxf(fmaf(sc.z, v[j].z, sh.z), 0.f); o.w = fmaxf(fmaf(sc.w, v[j].w, sh.w), 0.f);
            st4(a + row * C + c, o);
        }
    }
    stamp_end(stamp);
}

static int ew_grid(size_t n, int sm) {
    size_t g = (n + 255) / 256, cap = (size_t)sm * 8;
    return (int)(g < cap ? (g ? g : 1) : cap);
}
static int row_grid(size_t P, int C4, int sm, int per_sm);
template <class K> static int blocks_per_sm(K kernel) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, 256, 0) != cudaSuccess || n < 1) { cudaGetLastError(); n = 4; }
    return n > 8 ? 8 : n;
}

void bn_relu_apply(Exec &ex, Pair t, size_t P, BnRef bn, void *a, bool a_bf16) {
    if (ex.dry) return;
    const int C4 = t.C() / 4;
    static const int occ16 = blocks_per_sm(bn_relu_apply_kernel<bf16>), occ32 = blocks_per_sm(bn_relu_apply_kernel<float>);
    const int g = row_grid(P, C4, ex.ctx->sm_count, a_bf16 ? occ16 : occ32);
    unsigned long long *stamp = ex.stamp_slot();
    if (a_bf16) launch(ex, bn_relu_apply_kernel<bf16>, g, 256, 0, t, P, C4, bn, (bf16 *)a, stamp);
    else launch(ex, bn_relu_apply_kernel<float>, g, 256, 0, t, P, C4, bn, (float *)a, stamp);
    ex.check("bn_relu_apply", (double)P * t.C() * (a_bf16 ? 6 : 8));
}

// dt = coef0*db - coef1 - coef2*xhat ; db = da*[scale*t+shift > 0]
// OUT 0: out[P,C] = dt (float or bf16) ; 1: outp = dt (fp32 pair) ; 2: outp = add + dt
// CAST (OUT 1, 2): also write the result as one bf16 [P,C] tensor
// A thread keeps one channel quad (its coefficients stay in registers) and strides the rows, four
// rows in flight; row_step = threads of the grid / C4 (the launch makes that a whole number).
template <class TO, int OUT, bool CAST>
__global__ void __launch_bounds__(256, 2) bn_relu_bwd_apply_kernel(const float *__restrict__ da, Pair t, size_t P, int C4, BnRef bn,
                                         const float *__restrict__ coef, TO *__restrict__ out, Pair add, Pair outp,
                                         bf16 *__restrict__ cast, unsigned long long *stamp) {
    pdl_enter();
    stamp_begin(stamp);
    const int C = C4 * 4;
    const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, nth = (size_t)gridDim.x * blockDim.x;
    const int q = (int)(gtid % C4), c = q * 4;
    const size_t row0 = gtid / C4, row_step = nth / C4;
    float4 sc, sh, mu, rs;
    bn_coef4(bn, c, sc, sh, mu, rs);
    const float4 k0 = ld4(coef + c), k1 = ld4(coef + C + c), k2 = ld4(coef + 2 * C + c);
    for (size_t rb = row0; rb < P; rb += 4 * row_step) {
        // all loads of the four rows leave before anything waits on one: rows beyond the end read the last row again and
        // are not stored
        float4 v[4], g[4], pa[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const size_t row = rb + j * row_step, rr = row < P ? row : P - 1;
            v[j] = t.ld4_raw(rr, c); g[j] = ld4(da + rr * C + c);
            if (OUT == 2) pa[j] = add.ld4_raw(rr, c);
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const size_t row = rb + j * row_step;
            if (row >= P) continue;
            v[j] = t.from_raw(v[j]);
            if (OUT == 2) pa[j] = add.from_raw(pa[j]);
            float4 o;
            o.x = k0.x * (fmaf(sc.x, v[j].x, sh.x) > 0.f ? g[j].x : 0.f) - k1.x - k2.x * ((v[j].x - mu.x) * rs.x);
            o.y = k0.y * (fmaf(sc.y, v[j].y, sh.y) > 0.f ? g[j].y : 0.f) - k1.y - k2.y * ((v[j].y - mu.y) * rs.y);
            o.z = k0.z * (fmaf(sc.z, v[j].z, sh.z) > 0.f ? g[j].z : 0.f) - k1.z - k2.z * ((v[j].z - mu.z) * rs.z);
            o.w = k0.w * (fmaf(sc.w, v[j].w, sh.w) > 0.f ? g[j].w : 0.f) - k1.w - k2.w * ((v[j].w - mu.w) * rs.w);
            if (OUT == 2) { o.x += pa[j].x; o.y += pa[j].y; o.z += pa[j].z; o.w += pa[j].w; }
            if (OUT == 0) st4(out + row * C + c, o);
            else st4(outp.at(row, c), o);
            if (CAST) st4(cast + row * C + c, o);
        }
    }
    stamp_end(stamp);
}

// grid for the row-strided elementwise kernels: 256 threads per block, a thread count that is a multiple of C4
// per_sm: blocks of the kernel that fit an SM at once (its occupancy): a grid of exactly the resident blocks, each
// striding over its share of the rows, has no partly filled last wave
static int row_grid(size_t P, int C4, int sm, int per_sm) {
    // smallest block count g >= wanted with (g * 256) % C4 == 0: C4 divides 256 * g when g is a multiple of C4 / gcd(C4, 256)
    int a = C4, b = 256;
    while (b) { int r = a % b; a = b; b = r; }
    const int unit = C4 / a;
    size_t want = (P * C4 + 1023) / 1024, cap = (size_t)sm * per_sm;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    return (int)((want + unit - 1) / unit * unit);
}

void bn_relu_bwd(Exec &ex, const float *da, Pair t, size_t P, BnRef bn, float *dgamma, float *dbeta, float *coef,
                 bool sums_done, void *out_single, bool out_bf16, Pair add, Pair out_pair, bf16 *out_cast) {
    const int C = t.C(), C4 = C / 4;
    RedShape r = red_shape(P, C, ex.ctx->sm_count);
    size_t m = ex.ws.mark();
    float *part = sums_done ? nullptr : ex.ws.get<float>((size_t)r.chunks * 2 * C);
    if (!ex.dry) {
        if (!sums_done) {
            dim3 grid(r.chunks, r.slabs), block(r.SW, r.RPP);
            launch(ex, col_reduce_kernel<1>, grid, block, (size_t)r.SW * r.RPP * 32, t, da, P, r.rows_per_cta, bn, part);
            ex.check("bn_bwd_partial", (double)P * C * 8);
            launch(ex, bn_bwd_finalize, cdiv((size_t)C * 32, 128), 128, 0, part, r.chunks, C, 1.0 / (double)P, bn.gamma, bn.rstd, dgamma, dbeta, coef);
            ex.check("bn_bwd_finalize");
        }
        static const int occ = blocks_per_sm(bn_relu_bwd_apply_kernel<float, 2, true>);      // the heaviest variant
        const int g = row_grid(P, C4, ex.ctx->sm_count, occ);
#define RV_ARGS da, t, P, C4, bn, coef
        unsigned long long *stamp = ex.stamp_slot();
        if (out_pair.p0 && add.p0) {
            if (out_cast) launch(ex, bn_relu_bwd_apply_kernel<float, 2, true>, g, 256, 0, RV_ARGS, nullptr, add, out_pair, out_cast, stamp);
            else launch(ex, bn_relu_bwd_apply_kernel<float, 2, false>, g, 256, 0, RV_ARGS, nullptr, add, out_pair, nullptr, stamp);
        } else if (out_pair.p0) {
            if (out_cast) launch(ex, bn_relu_bwd_apply_kernel<float, 1, true>, g, 256, 0, RV_ARGS, nullptr, add, out_pair, out_cast, stamp);
            else launch(ex, bn_relu_bwd_apply_kernel<float, 1, false>, g, 256, 0, RV_ARGS, nullptr, add, out_pair, nullptr, stamp);
        } else if (out_bf16) launch(ex, bn_relu_bwd_apply_kernel<bf16, 0, false>, g, 256, 0, RV_ARGS, (bf16 *)out_single, add, out_pair, nullptr, stamp);
        else launch(ex, bn_relu_bwd_apply_kernel<float, 0, false>, g, 256, 0, RV_ARGS, (float *)out_single, add, out_pair, nullptr, stamp);
#undef RV_ARGS
        ex.check("bn_relu_bwd_apply", (double)P * C * ((out_pair.p0 ? (add.p0 ? 16 : 12) : (out_bf16 ? 10 : 12)) + (out_cast ? 2 : 0)));
    }
    ex.ws.release(m);
}

template <class TO>
__global__ void concat_cast_kernel(Pair src, size_t nquads, int C4, TO *__restrict__ dst) {
    pdl_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nquads; i += (size_t)gridDim.x * blockDim.x) {
        size_t row = i / C4; int q = (int)(i - row * C4);
        st4(dst + i * 4, src.ld4(row, q * 4));
    }
}

void concat_cast(Exec &ex, Pair src, size_t P, void *dst, bool dst_bf16) {
    if (ex.dry) return;
    const int C4 = src.C() / 4; size_t nq = P * C4; int g = ew_grid(nq, ex.ctx->sm_count);
    if (dst_bf16) launch(ex, concat_cast_kernel<bf16>, g, 256, 0, src, nq, C4, (bf16 *)dst);
    else launch(ex, concat_cast_kernel<float>, g, 256, 0, src, nq, C4, (float *)dst);
    ex.check("concat_cast", (double)P * src.C() * (dst_bf16 ? 6 : 8));
}

// ------------------------------------------------------------------ max-pool 3x3 stride 2 pad 1 (NHWC)
__global__ void maxpool_fwd_kernel(const float *__restrict__ in, float *__restrict__ out, int N, int H, int W, int C4, int Ho, int Wo) {
    pdl_enter();
    size_t n = (size_t)N * Ho * Wo * C4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        int q = (int)(i % C4); size_t p = i / C4;
        int j = (int)(p % Wo); p /= Wo; int io = (int)(p % Ho); int b = (int)(p / Ho);
        float4 m = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        for (int kh = 0; kh < 3; kh++) for (int kw = 0; kw < 3; kw++) {
            int y = io * 2 + kh - 1, x = j * 2 + kw - 1;
            if (y < 0 || y >= H || x < 0 || x >= W) continue;
            float4 v = ld4(in + (((size_t)b * H + y) * W + x) * C4 * 4 + q * 4);
            m.x = fmaxf(m.x, v.x); m.y = fmaxf(m.y, v.y); m.z = fmaxf(m.z, v.z); m.w = fmaxf(m.w, v.w);
        }
        st4(out + i * 4, m);
    }
}

// Gradient goes to the first maximum met in (kh,kw) row-major scan of each window.
// A CTA takes 8 x 8 input pixels x 8 channel quads of one image: it loads them with the halo their windows reach
// (11 x 11 pixels; outside the image: -inf) and the 5 x 5 gradients of those windows into shared memory, finds
// every window's first maximum once, and each input element then asks its (at most four) windows whether it is
// theirs -- one global read per element instead of one per window tap.
__global__ void __launch_bounds__(256) maxpool_bwd_kernel(const float *__restrict__ in, const float *__restrict__ dout, float *__restrict__ din,
                                                          int N, int H, int W, int C4, int Ho, int Wo, int tiles_y, int tiles_x, int tiles_q) {
    pdl_enter();
    __shared__ float4 tin[11 * 11 * 8];
    __shared__ float4 tg[5 * 5 * 8];
    __shared__ int4 tam[5 * 5 * 8];
    int t = blockIdx.x;
    const int tq = t % tiles_q; t /= tiles_q;
    const int tx = t % tiles_x; t /= tiles_x;
    const int ty = t % tiles_y; const int b = t / tiles_y;
    const int y0 = ty * 8, x0 = tx * 8, q0 = tq * 8;
    const int tid = threadIdx.x;
    const float ninf = -INFINITY;
    for (int idx = tid; idx < 11 * 11 * 8; idx += 256) {
        const int q = idx & 7, pos = idx >> 3, ry = pos / 11, rx = pos - ry * 11;
        const int yy = y0 - 1 + ry, xx = x0 - 1 + rx;
        float4 v = make_float4(ninf, ninf, ninf, ninf);
        if (yy >= 0 && yy < H && xx >= 0 && xx < W && q0 + q < C4) v = ld4(in + ((((size_t)b * H + yy) * W + xx) * C4 + q0 + q) * 4);
        tin[idx] = v;
    }
    if (tid < 5 * 5 * 8) {
        const int q = tid & 7, wpos = tid >> 3, wi = wpos / 5, wj = wpos - wi * 5;
        const int io = y0 / 2 + wi, j = x0 / 2 + wj;
        float4 g = make_float4(0.f, 0.f, 0.f, 0.f);
        if (io < Ho && j < Wo && q0 + q < C4) g = ld4(dout + ((((size_t)b * Ho + io) * Wo + j) * C4 + q0 + q) * 4);
        tg[tid] = g;
    }
    __syncthreads();
    if (tid < 5 * 5 * 8) {
        // window (wi, wj) covers tile rows 2wi .. 2wi+2, columns 2wj .. 2wj+2
        const int q = tid & 7, wpos = tid >> 3, wi = wpos / 5, wj = wpos - wi * 5;
        float4 best = make_float4(ninf, ninf, ninf, ninf);
        int4 at = make_int4(-1, -1, -1, -1);
        for (int kh = 0; kh < 3; kh++)
            for (int kw = 0; kw < 3; kw++) {
                const int pos = (2 * wi + kh) * 11 + 2 * wj + kw;
                const float4 v = tin[pos * 8 + q];
                if (v.x > best.x) { best.x = v.x; at.x = pos; }
                if (v.y > best.y) { best.y = v.y; at.y = pos; }
                if (v.z > best.z) { best.z = v.z; at.z = pos; }
                if (v.w > best.w) { best.w = v.w; at.w = pos; }
            }
        tam[tid] = at;
    }
    __syncthreads();
    for (int idx = tid; idx < 8 * 8 * 8; idx += 256) {
        const int q = idx & 7, lp = idx >> 3, ly = lp >> 3, lx = lp & 7;
        const int y = y0 + ly, x = x0 + lx;
        if (y >= H || x >= W || q0 + q >= C4) continue;
        const int mine = (ly + 1) * 11 + lx + 1;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int wi = ly / 2; wi <= (ly + 1) / 2; wi++)
            for (int wj = lx / 2; wj <= (lx + 1) / 2; wj++) {
                const int w = (wi * 5 + wj) * 8 + q;        // windows beyond the pooled image carry a zero gradient
                const int4 at = tam[w];
                const float4 g = tg[w];
                if (at.x == mine) acc.x += g.x;
                if (at.y == mine) acc.y += g.y;
                if (at.z == mine) acc.z += g.z;
                if (at.w == mine) acc.w += g.w;
            }
        st4(din + ((((size_t)b * H + y) * W + x) * C4 + q0 + q) * 4, acc);
    }
}

void maxpool_fwd(Exec &ex, const float *in, float *out, int N, int H, int W, int C) {
    if (ex.dry) return;
    int Ho = conv_out(H, 3, 2), Wo = conv_out(W, 3, 2);
    size_t n = (size_t)N * Ho * Wo * (C / 4);
    launch(ex, maxpool_fwd_kernel, ew_grid(n, ex.ctx->sm_count), 256, 0, in, out, N, H, W, C / 4, Ho, Wo);
    ex.check("maxpool_fwd");
}
void maxpool_bwd(Exec &ex, const float *in, const float *dout, float *din, int N, int H, int W, int C) {
    if (ex.dry) return;
    int Ho = conv_out(H, 3, 2), Wo = conv_out(W, 3, 2);
    const int C4 = C / 4, tiles_y = (H + 7) / 8, tiles_x = (W + 7) / 8, tiles_q = (C4 + 7) / 8;
    launch(ex, maxpool_bwd_kernel, (unsigned)((size_t)N * tiles_y * tiles_x * tiles_q), 256, 0, in, dout, din, N, H, W, C4, Ho, Wo, tiles_y, tiles_x, tiles_q);
    ex.check("maxpool_bwd");
}

// ------------------------------------------------------------------ head: avgpool -> FC -> softmax CE -> argmax
__global__ void avgpool_kernel(Pair y, int HW, float *__restrict__ feat) {
    pdl_enter();
    extern __shared__ float4 sm4[];
    const int C = y.C(), C4 = C / 4, SW = blockDim.x, RPP = blockDim.y;
    const int q = blockIdx.y * SW + threadIdx.x, n = blockIdx.x;
    const bool valid = q < C4;
    float4 s = make_float4(0, 0, 0, 0);
    if (valid)
        for (int r = threadIdx.y; r < HW; r += RPP) {
            float4 v = y.ld4((size_t)n * HW + r, q * 4);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
    sm4[threadIdx.y * SW + threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y == 0 && valid) {
        for (int yy = 1; yy < RPP; yy++) { float4 a = sm4[yy * SW + threadIdx.x]; s.x += a.x; s.y += a.y; s.z += a.z; s.w += a.w; }
        float inv = 1.f / (float)HW;
        s.x *= inv; s.y *= inv; s.z *= inv; s.w *= inv;
        st4(feat + (size_t)n * C + q * 4, s);
    }
}

// one warp per (n,k)
__global__ void fc_fwd_kernel(const float *__restrict__ feat, const float *__restrict__ Wfc, const float *__restrict__ bfc,
                              int N, int C, int K, float *__restrict__ logits) {
    pdl_enter();
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= N * K) return;
    int n = warp / K, k = warp - n * K;
    float s = 0.f;
    for (int c = lane; c < C; c += 32) s = fmaf(feat[(size_t)n * C + c], Wfc[(size_t)k * C + c], s);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) logits[warp] = s + bfc[k];
}

// one warp per sample: stable log-sum-exp, dlogits = (softmax - onehot)/N, arg-max (lowest index on ties)
// A label outside [0, K) is reported, not followed: nothing is read at it, the sample's loss becomes NaN and the
// context's status word is set to REVNET_E_INVALID_ARG (revnet_check_device returns it).
__global__ void softmax_ce_kernel(const float *__restrict__ logits, const int32_t *__restrict__ labels, int N, int K,
                                  float *__restrict__ dlogits, float *__restrict__ loss_n, int32_t *__restrict__ pred, int *status) {
    pdl_enter();
    int n = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (n >= N) return;
    const float *z = logits + (size_t)n * K;
    float m = -INFINITY; int mi = 0x7fffffff;
    for (int k = lane; k < K; k += 32) { float v = z[k]; if (v > m) { m = v; mi = k; } }
    for (int o = 16; o; o >>= 1) {
        float om = __shfl_xor_sync(0xffffffffu, m, o); int oi = __shfl_xor_sync(0xffffffffu, mi, o);
        if (om > m || (om == m && oi < mi)) { m = om; mi = oi; }
    }
    float s = 0.f;
    for (int k = lane; k < K; k += 32) s += expf(z[k] - m);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const int lab = labels[n];
    const bool lab_ok = lab >= 0 && lab < K;
    const float inv = 1.f / s, invN = 1.f / (float)N;
    for (int k = lane; k < K; k += 32) dlogits[(size_t)n * K + k] = (expf(z[k] - m) * inv - (k == lab ? 1.f : 0.f)) * invN;
    if (lane == 0) {
        loss_n[n] = lab_ok ? m + logf(s) - z[lab] : __int_as_float(0x7fc00000);
        pred[n] = mi;
        if (!lab_ok && status) atomicCAS(status, 0, (int)REVNET_E_INVALID_ARG);
    }
}

__global__ void mean_kernel(const float *__restrict__ v, int N, float *out) {
    pdl_enter();
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double s = 0; for (int i = 0; i < N; i++) s += v[i];
        *out = (float)(s / N);
    }
}

void head_fwd(Exec &ex, Pair y, int N, int HW, const float *Wfc, const float *bfc, const int32_t *labels,
              int K, float *feat, float *logits, float *dlogits, float *loss, int32_t *pred) {
    const int C = y.C();
    ex.flops += 2ull * N * C * K;
    size_t m = ex.ws.mark();
    float *loss_n = ex.ws.get<float>(N);
    if (!ex.dry) {
        int C4 = C / 4, SW = C4 < 128 ? C4 : 128, RPP = 256 / SW; if (RPP < 1) RPP = 1;
        dim3 grid(N, cdiv(C4, SW)), block(SW, RPP);
        launch(ex, avgpool_kernel, grid, block, (size_t)SW * RPP * 16, y, HW, feat);
        ex.check("avgpool");
        launch(ex, fc_fwd_kernel, cdiv((size_t)N * K * 32, 256), 256, 0, feat, Wfc, bfc, N, C, K, logits);
        ex.check("fc_fwd");
        launch(ex, softmax_ce_kernel, cdiv((size_t)N * 32, 256), 256, 0, logits, labels, N, K, dlogits, loss_n, pred, ex.ctx->dev_status);
        ex.check("softmax_ce");
        launch(ex, mean_kernel, 1, 32, 0, loss_n, N, loss);
        ex.check("loss_mean");
    }
    ex.ws.release(m);
}

__global__ void fc_wgrad_kernel(const float *__restrict__ dlogits, const float *__restrict__ feat, int N, int C, int K,
                                float *__restrict__ dW, float *__restrict__ db) {
    pdl_enter();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < (size_t)K * C) {
        int k = (int)(i / C), c = (int)(i - (size_t)k * C);
        float s = 0.f;
        for (int n = 0; n < N; n++) s = fmaf(dlogits[(size_t)n * K + k], feat[(size_t)n * C + c], s);
        dW[i] = s;
    }
    if (i < (size_t)K) { float s = 0.f; for (int n = 0; n < N; n++) s += dlogits[(size_t)n * K + i]; db[i] = s; }
}
// the same for a small layer: one warp per element of dW (and of db), lanes over the samples, added by a shuffle tree
__global__ void fc_wgrad_warp_kernel(const float *__restrict__ dlogits, const float *__restrict__ feat, int N, int C, int K,
                                     float *__restrict__ dW, float *__restrict__ db) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const size_t w = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const size_t n_out = (size_t)K * C + K;
    if (w >= n_out) return;
    float s = 0.f;
    if (w < (size_t)K * C) {
        const int k = (int)(w / C), c = (int)(w - (size_t)k * C);
        for (int n = lane; n < N; n += 32) s = fmaf(dlogits[(size_t)n * K + k], feat[(size_t)n * C + c], s);
    } else {
        const int k = (int)(w - (size_t)K * C);
        for (int n = lane; n < N; n += 32) s += dlogits[(size_t)n * K + k];
    }
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) { if (w < (size_t)K * C) dW[w] = s; else db[w - (size_t)K * C] = s; }
}
__global__ void fc_dgrad_kernel(const float *__restrict__ dlogits, const float *__restrict__ Wfc, int N, int C, int K,
                                float scale, float *__restrict__ dfeat) {
    pdl_enter();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)N * C) return;
    int n = (int)(i / C), c = (int)(i - (size_t)n * C);
    float s = 0.f;
    for (int k = 0; k < K; k++) s = fmaf(dlogits[(size_t)n * K + k], Wfc[(size_t)k * C + c], s);
    dfeat[i] = s * scale;
}
__global__ void avgpool_bwd_kernel(const float *__restrict__ dfeat, Pair dy, size_t nquads, int C4, int HW) {
    pdl_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nquads; i += (size_t)gridDim.x * blockDim.x) {
        size_t row = i / C4; int q = (int)(i - row * C4); size_t n = row / HW;
        st4(dy.at(row, q * 4), ld4(dfeat + n * C4 * 4 + q * 4));
    }
}

void head_bwd(Exec &ex, Pair dy, int N, int HW, const float *Wfc, const float *feat, const float *dlogits,
              int K, float *dWfc, float *dbfc, float *dfeat) {
    const int C = dy.C();
    ex.flops += 4ull * N * C * K;
    if (ex.dry) return;
    if ((size_t)K * C <= 65536) launch(ex, fc_wgrad_warp_kernel, cdiv(((size_t)K * C + K) * 32, 256), 256, 0, dlogits, feat, N, C, K, dWfc, dbfc);
    else launch(ex, fc_wgrad_kernel, cdiv((size_t)K * C, 256), 256, 0, dlogits, feat, N, C, K, dWfc, dbfc);
    ex.check("fc_wgrad");
    launch(ex, fc_dgrad_kernel, cdiv((size_t)N * C, 256), 256, 0, dlogits, Wfc, N, C, K, 1.f / (float)HW, dfeat);
    ex.check("fc_dgrad");
    size_t nq = (size_t)N * HW * (C / 4);
    launch(ex, avgpool_bwd_kernel, ew_grid(nq, ex.ctx->sm_count), 256, 0, dfeat, dy, nq, C / 4, HW);
    ex.check("avgpool_bwd");
}

// ------------------------------------------------------------------ shortcut of a down-sampling unit
// S(x): 2x2 average pooling with stride 2, then zero channels up to cout; x and S(x) in the coupling-state format
// (on a fixed-point state the mean of the four grid values is rounded to the grid, ties to even).
__global__ void shortcut_fwd_kernel(const float *__restrict__ x, float *__restrict__ out, int N, int H, int W, int cin, int cout, float q) {
    pdl_enter();
    const int Ho = H >> 1, Wo = W >> 1, C4 = cout >> 2;
    const size_t n = (size_t)N * Ho * Wo * C4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % C4) * 4; size_t p = i / C4;
        const int xo = (int)(p % Wo); p /= Wo;
        const int yo = (int)(p % Ho); const size_t b = p / Ho;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < cin) {
            const float *s0 = x + (((b * H + 2 * yo) * W + 2 * xo) * (size_t)cin + c);
            const float *s1 = s0 + (size_t)W * cin;
            if (q == 0.f) {
                const float4 a = ld4(s0), bq = ld4(s0 + cin), cq = ld4(s1), d = ld4(s1 + cin);
                o = make_float4((a.x + bq.x + cq.x + d.x) * 0.25f, (a.y + bq.y + cq.y + d.y) * 0.25f,
                                (a.z + bq.z + cq.z + d.z) * 0.25f, (a.w + bq.w + cq.w + d.w) * 0.25f);
            } else {
                const int4 a = *reinterpret_cast<const int4 *>(s0), bq = *reinterpret_cast<const int4 *>(s0 + cin);
                const int4 cq = *reinterpret_cast<const int4 *>(s1), d = *reinterpret_cast<const int4 *>(s1 + cin);
                auto avg = [](int u, int v, int w, int z) {
                    const int sum = u + v + w + z;
                    int k = sum >> 2; const int r = sum & 3;             // floor and remainder (in quarters)
                    if (r == 3 || (r == 2 && (k & 1))) k++;              // nearest, ties to even
                    return __int_as_float(k);
                };
                o = make_float4(avg(a.x, bq.x, cq.x, d.x), avg(a.y, bq.y, cq.y, d.y), avg(a.z, bq.z, cq.z, d.z), avg(a.w, bq.w, cq.w, d.w));
            }
        }
        st4(out + i * 4, o);
    }
}
// S^T d: the first cin channels of d [N, H/2, W/2, cout], each value spread over its 2x2 window with weight 1/4 -> [N, H, W, cin]
__global__ void shortcut_bwd_kernel(const float *__restrict__ d, float *__restrict__ gx, int N, int H, int W, int cin, int cout) {
    pdl_enter();
    const int Ho = H >> 1, Wo = W >> 1, C4 = cin >> 2;
    const size_t n = (size_t)N * H * W * C4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % C4) * 4; size_t p = i / C4;
        const int xx = (int)(p % W); p /= W;
        const int yy = (int)(p % H); const size_t b = p / H;
        const float4 v = ld4(d + (((b * Ho + (yy >> 1)) * Wo + (xx >> 1)) * (size_t)cout + c));
        st4(gx + i * 4, make_float4(v.x * 0.25f, v.y * 0.25f, v.z * 0.25f, v.w * 0.25f));
    }
}
void shortcut_fwd(Exec &ex, const float *x, float *out, int N, int H, int W, int cin, int cout, float q) {
    if (ex.dry) return;
    const size_t n = (size_t)N * (H / 2) * (W / 2) * (cout / 4);
    launch(ex, shortcut_fwd_kernel, ew_grid(n, ex.ctx->sm_count), 256, 0, x, out, N, H, W, cin, cout, q);
    ex.check("shortcut_fwd", (double)N * H * W * cin * 4 + (double)n * 16);
}
void shortcut_bwd(Exec &ex, const float *d, float *gx, int N, int H, int W, int cin, int cout) {
    if (ex.dry) return;
    const size_t n = (size_t)N * H * W * (cin / 4);
    launch(ex, shortcut_bwd_kernel, ew_grid(n, ex.ctx->sm_count), 256, 0, d, gx, N, H, W, cin, cout);
    ex.check("shortcut_bwd", (double)n * 16 * 1.25);
}

// ------------------------------------------------------------------ SGD with momentum and weight decay
// v <- mu v + (g + wd w [decayed segments only]); w <- w - lr v   (Appendix 6.1).  Four floats per access, four
// accesses in flight per thread; every segment but the last starts and ends on a multiple of four floats (channel
// counts are multiples of four), so a quad lies in one segment; the floats behind the last whole quad go one by one.
__device__ __forceinline__ int sgd_segment(const uint32_t *__restrict__ seg_end, int n_seg, size_t i) {
    int lo = 0, hi = n_seg - 1;                  // first segment whose end is > i
    while (lo < hi) { int mid = (lo + hi) >> 1; if (seg_end[mid] > i) hi = mid; else lo = mid + 1; }
    return lo;
}
__global__ void __launch_bounds__(256) sgd_kernel(float *__restrict__ p, const float *__restrict__ g, float *__restrict__ v, size_t n,
                                                  const uint32_t *__restrict__ seg_end, const uint8_t *__restrict__ seg_decay, int n_seg,
                                                  float lr, float mu, float wd) {
    pdl_enter();
    const size_t n4 = n >> 2, stride = (size_t)gridDim.x * blockDim.x;
    float4 *p4 = reinterpret_cast<float4 *>(p), *v4 = reinterpret_cast<float4 *>(v);
    const float4 *g4 = reinterpret_cast<const float4 *>(g);
    for (size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < n4; i0 += 4 * stride) {
        float4 w[4], gg[4], vv[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const size_t i = i0 + j * stride;
            if (i < n4) { w[j] = p4[i]; gg[j] = g4[i]; vv[j] = v4[i]; }
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const size_t i = i0 + j * stride;
            if (i >= n4) continue;
            const float d = seg_decay[sgd_segment(seg_end, n_seg, i * 4)] ? wd : 0.f;
            float4 o;
            o.x = fmaf(mu, vv[j].x, gg[j].x + d * w[j].x); o.y = fmaf(mu, vv[j].y, gg[j].y + d * w[j].y);
            o.z = fmaf(mu, vv[j].z, gg[j].z + d * w[j].z); o.w = fmaf(mu, vv[j].w, gg[j].w + d * w[j].w);
            v4[i] = o;
            p4[i] = make_float4(w[j].x - lr * o.x, w[j].y - lr * o.y, w[j].z - lr * o.z, w[j].w - lr * o.w);
        }
    }
    if (blockIdx.x == 0)
        for (size_t i = n4 * 4 + threadIdx.x; i < n; i += blockDim.x) {
            const float w = p[i];
            const float gg = g[i] + (seg_decay[sgd_segment(seg_end, n_seg, i)] ? wd * w : 0.f);
            const float vv = fmaf(mu, v[i], gg);
            v[i] = vv;
            p[i] = w - lr * vv;
        }
}
// the same, one float at a time: for a parameter layout in which some segment does not start on a multiple of four
__global__ void sgd_scalar_kernel(float *__restrict__ p, const float *__restrict__ g, float *__restrict__ v, size_t n,
                                  const uint32_t *__restrict__ seg_end, const uint8_t *__restrict__ seg_decay, int n_seg,
                                  float lr, float mu, float wd) {
    pdl_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float w = p[i];
        const float gg = g[i] + (seg_decay[sgd_segment(seg_end, n_seg, i)] ? wd * w : 0.f);
        const float vv = fmaf(mu, v[i], gg);
        v[i] = vv;
        p[i] = w - lr * vv;
    }
}
void sgd_update(Exec &ex, float *params, const float *grads, float *mom, size_t n, const uint32_t *seg_end,
                const uint8_t *seg_decay, int n_seg, float lr, float momentum, float wd, bool quad_aligned) {
    if (ex.dry) return;
    if (quad_aligned) launch(ex, sgd_kernel, ew_grid(n / 16 + 1, ex.ctx->sm_count), 256, 0, params, grads, mom, n, seg_end, seg_decay, n_seg, lr, momentum, wd);
    else launch(ex, sgd_scalar_kernel, ew_grid(n, ex.ctx->sm_count), 256, 0, params, grads, mom, n, seg_end, seg_decay, n_seg, lr, momentum, wd);
    ex.check("sgd", (double)n * 20);
}

__global__ void max_abs_diff_kernel(const float *__restrict__ a, const float *__restrict__ b, size_t n, float q, float *out) {
    pdl_enter();
    float m = 0.f;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        if (q == 0.f) m = fmaxf(m, fabsf(a[i] - b[i]));
        else m = fmaxf(m, fabsf((float)(reinterpret_cast<const int *>(a)[i] - reinterpret_cast<const int *>(b)[i])) * q);
    }
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<int *>(out), __float_as_int(m));   // m >= 0
}
void max_abs_diff(Exec &ex, const float *a, const float *b, size_t n, float q, float *out) {
    if (ex.dry) return;
    launch(ex, max_abs_diff_kernel, ew_grid(n, ex.ctx->sm_count), 256, 0, a, b, n, q, out);
    ex.check("max_abs_diff");
}
void fill_zero(Exec &ex, void *p, size_t bytes) {
    if (ex.dry) return;
    cudaMemsetAsync(p, 0, bytes, ex.stream);
}

__global__ void upsample_zero_kernel(const uint4 *__restrict__ in, uint4 *__restrict__ out, int N, int Ho, int Wo, int C8) {
    pdl_enter();
    const size_t n = (size_t)N * Ho * 2 * Wo * 2 * C8;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % C8); size_t p = i / C8;
        const int x = (int)(p % (2 * Wo)); p /= 2 * Wo;
        const int y = (int)(p % (2 * Ho)); const size_t b = p / (2 * Ho);
        uint4 v = make_uint4(0, 0, 0, 0);
        if (!(x & 1) && !(y & 1)) v = in[((b * Ho + (y >> 1)) * Wo + (x >> 1)) * C8 + c];
        out[i] = v;
    }
}
void upsample_zero_bf16(Exec &ex, const bf16 *in, bf16 *out, int N, int Ho, int Wo, int C) {
    if (ex.dry) return;
    const size_t n = (size_t)N * Ho * 2 * Wo * 2 * (C / 8);
    launch(ex, upsample_zero_kernel, ew_grid(n, ex.ctx->sm_count), 256, 0, (const uint4 *)in, (uint4 *)out, N, Ho, Wo, C / 8);
    ex.check("upsample_zero", (double)n * 16 * 1.25);
}
