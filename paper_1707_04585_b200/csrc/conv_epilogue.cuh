// Epilogue shared by the tensor-core convolution kernels: drains a 128-row accumulator from tensor
// memory through a padded shared-memory stage, so that global accesses are coalesced, and fuses
//   - the coupling  y = x + F  /  x = y - F  on the float or fixed-point state      (Section 3.1)
//   - per-channel sums of the stored result (the batch statistics of the BN that reads it next,
//     Eq. 2: a(x) = ReLU(BN(x))), or, for a data gradient, the two sums of the BN+ReLU backward
//   - the reduction of those sums over the grid: the CTA that finishes last adds the per-CTA
//     partials in a fixed order (double precision) and writes mean / 1/sqrt(var+eps), or
//     dgamma, dbeta and the coefficients of the BN-backward formula.
// Everything is summed in an order fixed by the launch shape, so a residual function recomputed
// in the backward pass reproduces its forward bits.
#pragma once
#include "common.cuh"
#include "tc_ptx.cuh"

namespace tc {

enum { EPI_PLAIN = 0, EPI_COUPLE = 1, EPI_BNBWD = 2 };

struct EpiArgs {
    int mode;
    Pair out, partner;       // [P, n_cols]; partner only with EPI_COUPLE
    int sign;                // EPI_COUPLE: +1 / -1
    int n_cols;              // valid output channels
    int pitch;               // floats per staged row: min(N tile, 64) + 4
    // reductions (optional: part == nullptr switches them off; EPI_BNBWD always reduces)
    float *part;             // [gridDim.x][n_cols/4][2][4]: per channel quad, 4 sums then 4 second sums
    unsigned int *counter;   // zero on entry, left zero
    double inv_count;        // 1 / pixels
    float eps;
    float *mean, *rstd;      // EPI_PLAIN / EPI_COUPLE: statistics of the stored result
    // EPI_BNBWD: the accumulator is da, the gradient w.r.t. a = ReLU(BN(t))
    Pair t;
    BnRef bn;
    float *dgamma, *dbeta, *coef;   // coef: [3][n_cols] = gamma*rstd, gamma*rstd*dbeta/M, gamma*rstd*dgamma/M
};

// Geometry of the 128-row tiles: a tile is BIMG images x BH rows x W columns of the OUTPUT.
struct TileGeom {
    int N, H, W;
    int BH, BIMG;
    int tiles_per_img;       // BIMG == 1
    int n_px_tiles;
    int hw_order;            // accumulator rows run (h, img, x) with x < Wp instead of (img, h, w)
    int Wp;                  // hw_order: row pitch in pixels (W rounded up to a multiple of 8); columns >= W are padding
};
__device__ __forceinline__ void tile_origin(const TileGeom &g, int t, int &n0, int &h0) {
    if (g.BIMG > 1) { n0 = t * g.BIMG; h0 = 0; }
    else { n0 = t / g.tiles_per_img; h0 = (t - n0 * g.tiles_per_img) * g.BH; }
}
constexpr int kEpiChunk = 64;                    // accumulator columns staged at a time
constexpr int kEpiPitch = kEpiChunk + 4;         // floats per staged row (bank-conflict padding)
constexpr int kEpiMaxChunks = 2;                 // N tile <= 128 columns
constexpr int kEpiSumFloats = kEpiMaxChunks * 128 * 8;   // per thread and chunk: 4 sums, 4 second sums
constexpr int kEpiStageBytes = 128 * kEpiPitch * 4;

__device__ __forceinline__ float4 ldcg4(const float *p) { return __ldcg(reinterpret_cast<const float4 *>(p)); }

// Which pixel an accumulator row holds depends on the tile only through its origin, so the part
// that does not is decoded once per CTA: rel = pixel offset relative to the tile's origin pixel
// (image n0, row h0, column 0), -1 for rows that are padding in every tile; hi = row | image << 16
// within the tile, for the bounds checks of ragged tiles.
struct RowMap { int rel[128]; int hi[128]; };
__device__ __forceinline__ void build_row_map(const TileGeom &g, RowMap *rm, int m) {
    int img, h, w;
    bool ok = true;
    if (g.hw_order) {
        w = m % g.Wp; img = (m / g.Wp) % g.BIMG; h = m / (g.BIMG * g.Wp);
        ok = w < g.W && h < g.BH;
    } else {
        ok = m < g.BIMG * g.BH * g.W;
        w = m % g.W; img = m / (g.BH * g.W); h = (m / g.W) % g.BH;
    }
    rm->rel[m] = ok ? (img * g.H + h) * g.W + w : -1;
    rm->hi[m] = h | (img << 16);
}
__device__ __forceinline__ int row_pixel(const RowMap *rm, const TileGeom &g, int n0, int h0, int tile_base, int row) {
    if (row >= 128) return -1;
    const int rel = rm->rel[row], hi = rm->hi[row];
    if (rel < 0 || h0 + (hi & 0xffff) >= g.H || n0 + (hi >> 16) >= g.N) return -1;
    return tile_base + rel;
}

// Shared memory of the epilogue: the padded stage (kEpiStageBytes) and each thread's running sums
// per column chunk (kEpiSumFloats floats, zeroed by epilogue_init).
__device__ __forceinline__ void epilogue_init(float *sums, int etid) {
    for (int i = etid; i < kEpiSumFloats; i += 128) sums[i] = 0.f;
}

// What the first four rows a thread handles read from global memory besides the accumulator (the
// partner of the coupling, or the BN input of a data gradient) can be fetched before the
// accumulator is complete.
struct EpiPrefetch { float4 v[4]; };
__device__ __forceinline__ void epilogue_prefetch(const EpiArgs &e, int BN, int col0, const RowMap *rm, const TileGeom &g,
                                                  int n0, int h0, int etid, EpiPrefetch &pre) {
    if (e.mode == EPI_PLAIN) return;
    const int cw = BN < kEpiChunk ? BN : kEpiChunk;
    const int QW = cw >> 2, rpp = 128 / QW;
    const int quad = etid % QW, r0 = etid / QW;
    const int col = col0 + quad * 4;
    const int tile_base = (n0 * g.H + h0) * g.W;
    if (r0 < rpp && col < e.n_cols) {
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const int pix = row_pixel(rm, g, n0, h0, tile_base, r0 + i * rpp);
            if (pix >= 0) {
                if (e.mode == EPI_COUPLE) pre.v[i] = *reinterpret_cast<const float4 *>(e.partner.at((size_t)pix, col));
                else pre.v[i] = e.t.ld4((size_t)pix, col);
            }
        }
    }
}

// One tile: 128 epilogue threads (etid 0..127; thread etid owns accumulator lane etid), BN
// accumulator columns starting at tensor-memory address tmem_acc; col0 = first output channel of
// this N tile.  rm and stage live in shared memory.  acc_empty is arrived on by every thread once
// the accumulator has been read.  The loops are deliberately not unrolled beyond four rows: the
// code has to stay small enough to live in the instruction cache.
__device__ __forceinline__ void epilogue_tile(const EpiArgs &e, uint32_t tmem_acc, int BN, int col0, const RowMap *rm,
                                              const TileGeom &g, int n0, int h0, float *stage, float *sums, int etid,
                                              uint64_t *acc_empty, const EpiPrefetch &pre) {
    const uint32_t lane_base = (uint32_t)((etid >> 5) * 32) << 16;
    const int tile_base = (n0 * g.H + h0) * g.W;
#pragma unroll 1
    for (int cc = 0; cc < BN; cc += kEpiChunk) {
        const int cw = BN - cc < kEpiChunk ? BN - cc : kEpiChunk;
        // phase 1: accumulator row -> staged row
#pragma unroll 1
        for (int c = 0; c < cw; c += 16) {
            float v[16];
            tmem_ld16(tmem_acc + lane_base + (uint32_t)(cc + c), v);
            float4 *dst = reinterpret_cast<float4 *>(stage + etid * e.pitch + c);
            dst[0] = make_float4(v[0], v[1], v[2], v[3]); dst[1] = make_float4(v[4], v[5], v[6], v[7]);
            dst[2] = make_float4(v[8], v[9], v[10], v[11]); dst[3] = make_float4(v[12], v[13], v[14], v[15]);
        }
        if (acc_empty && cc + cw >= BN) { tc_fence_before(); mbar_arrive(acc_empty); }
        named_barrier(1, 128);
        // phase 2: thread = (row r0 of each pass, channel quad); consecutive threads touch consecutive addresses
        const int QW = cw >> 2, rpp = 128 / QW;
        const int quad = etid % QW, r0 = etid / QW;
        const int col = col0 + cc + quad * 4;
        if (r0 < rpp && col < e.n_cols) {
            float4 sc = make_float4(0, 0, 0, 0), sh = sc, mu = sc, rs = sc;
            if (e.mode == EPI_BNBWD) bn_coef4(e.bn, col, sc, sh, mu, rs);
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f, q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
#pragma unroll 1
            for (int rb = r0; rb < 128; rb += 4 * rpp) {
                int pix[4]; float4 aux[4];
                const bool fetched = cc == 0 && rb == r0;
                // loads of the partner / BN input first: they may alias the stores below
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    pix[i] = row_pixel(rm, g, n0, h0, tile_base, rb + i * rpp);
                    if (pix[i] >= 0) {
                        if (fetched) aux[i] = pre.v[i];
                        else if (e.mode == EPI_COUPLE) aux[i] = *reinterpret_cast<const float4 *>(e.partner.at((size_t)pix[i], col));
                        else if (e.mode == EPI_BNBWD) aux[i] = e.t.ld4((size_t)pix[i], col);
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    if (pix[i] < 0) continue;
                    float4 v = *reinterpret_cast<const float4 *>(stage + (rb + i * rpp) * e.pitch + quad * 4);
                    if (e.mode == EPI_BNBWD) {
                        *reinterpret_cast<float4 *>(e.out.at((size_t)pix[i], col)) = v;
                        const float4 t = aux[i];
                        const float dx = fmaf(sc.x, t.x, sh.x) > 0.f ? v.x : 0.f, dy = fmaf(sc.y, t.y, sh.y) > 0.f ? v.y : 0.f;
                        const float dz = fmaf(sc.z, t.z, sh.z) > 0.f ? v.z : 0.f, dw = fmaf(sc.w, t.w, sh.w) > 0.f ? v.w : 0.f;
                        s0 += dx; s1 += dy; s2 += dz; s3 += dw;
                        q0 += dx * ((t.x - mu.x) * rs.x); q1 += dy * ((t.y - mu.y) * rs.y);
                        q2 += dz * ((t.z - mu.z) * rs.z); q3 += dw * ((t.w - mu.w) * rs.w);
                    } else {
                        if (e.mode == EPI_COUPLE) v = e.out.couple4_with((size_t)pix[i], col, v, aux[i], e.sign);
                        else v = e.out.store4((size_t)pix[i], col, v);
                        s0 += v.x; s1 += v.y; s2 += v.z; s3 += v.w;
                        q0 += v.x * v.x; q1 += v.y * v.y; q2 += v.z * v.z; q3 += v.w * v.w;
                    }
                }
            }
            if (e.part) {       // this thread's own slot: no other thread touches it
                float4 *slot = reinterpret_cast<float4 *>(sums + ((cc / kEpiChunk) * 128 + etid) * 8);
                float4 a = slot[0], b = slot[1];
                a.x += s0; a.y += s1; a.z += s2; a.w += s3; b.x += q0; b.y += q1; b.z += q2; b.w += q3;
                slot[0] = a; slot[1] = b;
            }
        }
        named_barrier(1, 128);
    }
}

// mean and 1 / sqrt(var + eps) from a channel's sum and second sum (double), rounded to float once
__device__ __forceinline__ void moments_of(double sum, double sum2, double inv_count, float eps, float &mean, float &rstd) {
    const double m = sum * inv_count;
    double var = sum2 * inv_count - m * m;
    if (var < 0) var = 0;
    mean = (float)m; rstd = (float)(1.0 / sqrt(var + (double)eps));
}

// Adds the per-CTA records of a reduction.  A record is 2C floats = C/2 float4 slots (per channel
// quad: sums, second sums); this call covers the slots slot0 .. slot0 + cw - 1 (cw <= 128, even).
// Thread = (slot, sub), slot fastest so that a warp reads whole records: it adds the records sub,
// sub + nsub, ... of its slot, ten loads in flight at a time; the subs are then added in order.
// (Giving a slot to consecutive lanes and adding them by shuffles was measured slower: the loads
// of a warp then touch 32 records.)  All in double precision, in an order that the number of
// records, cw and NT fix.  Result: tot[slot - slot0][4].  Called by NT threads (tid = 0..NT-1)
// that share named barrier 1; red: [NT][4] doubles, tot: [128][4] doubles of shared memory.
template <int NT>
__device__ __forceinline__ void reduce_records(const float *part, int parts, int C, int slot0, int cw, double *red, double *tot, int tid) {
    const int nsub = NT / cw;
    const int r = tid % cw, sub = tid / cw;
    if (sub < nsub) {
        double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
        const float *src = part + (size_t)(slot0 + r) * 4;
        constexpr int kInFlight = 10;
        for (int i = sub; i < parts; i += kInFlight * nsub) {
            float4 v[kInFlight];
#pragma unroll
            for (int k = 0; k < kInFlight; k++) {
                const int idx = i + k * nsub;
                v[k] = idx < parts ? ldcg4(src + (size_t)idx * 2 * C) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int k = 0; k < kInFlight; k++) { s0 += (double)v[k].x; s1 += (double)v[k].y; s2 += (double)v[k].z; s3 += (double)v[k].w; }
        }
        red[tid * 4] = s0; red[tid * 4 + 1] = s1; red[tid * 4 + 2] = s2; red[tid * 4 + 3] = s3;
    }
    named_barrier(1, NT);
    if (tid < cw) {
        double s0 = red[tid * 4], s1 = red[tid * 4 + 1], s2 = red[tid * 4 + 2], s3 = red[tid * 4 + 3];
        for (int y = 1; y < nsub; y++) {
            const double *o = red + (y * cw + tid) * 4;
            s0 += o[0]; s1 += o[1]; s2 += o[2]; s3 += o[3];
        }
        double *d = tot + tid * 4;
        d[0] = s0; d[1] = s1; d[2] = s2; d[3] = s3;
    }
    named_barrier(1, NT);
}

template <int NT>
__device__ __forceinline__ void epilogue_publish(const EpiArgs &e, float *scratch, int etid);

// After the last tile: per-CTA partials, grid-wide count, and the finalize by the CTA that comes last.
__device__ __forceinline__ void epilogue_finish(const EpiArgs &e, int BN, int col0, float *stage, const float *sums, int etid) {
    if (!e.part) return;
    float *scratch = stage;
    float *mine = e.part + (size_t)blockIdx.x * 2 * e.n_cols;
#pragma unroll 1
    for (int cc = 0; cc < BN; cc += kEpiChunk) {
        const int cw = BN - cc < kEpiChunk ? BN - cc : kEpiChunk;
        const int QW = cw >> 2, rpp = 128 / QW;
        const int quad = etid % QW, r0 = etid / QW;
        const int col = col0 + cc + quad * 4;
        if (r0 == 0 && col < e.n_cols) {
            const float *base = sums + (size_t)(cc / kEpiChunk) * 128 * 8;
            float r[8];
#pragma unroll
            for (int j = 0; j < 8; j++) r[j] = base[quad * 8 + j];
            for (int y = 1; y < rpp; y++)
#pragma unroll
                for (int j = 0; j < 8; j++) r[j] += base[(y * QW + quad) * 8 + j];
            *reinterpret_cast<float4 *>(mine + 2 * col) = make_float4(r[0], r[1], r[2], r[3]);
            *reinterpret_cast<float4 *>(mine + 2 * col + 4) = make_float4(r[4], r[5], r[6], r[7]);
        }
    }
    epilogue_publish<128>(e, scratch, etid);
}

// Once every CTA has written its partial record into e.part: count, and let the CTA that comes
// last reduce the records in a fixed order and write the results.  Called by NT threads (etid = 0..NT-1);
// scratch: (NT + 128) * 32 bytes of shared memory.
template <int NT>
__device__ __forceinline__ void epilogue_publish(const EpiArgs &e, float *scratch, int etid) {
    // publish, count, and let the last CTA of the grid reduce
    __threadfence();
    named_barrier(1, NT);
    unsigned int *flag = reinterpret_cast<unsigned int *>(scratch);
    if (etid == 0) {
        const unsigned int total = gridDim.x * gridDim.y;
        const unsigned int old = atomicAdd(e.counter, 1u);
        *flag = (old == total - 1) ? 1u : 0u;
    }
    named_barrier(1, NT);
    const bool last = *flag != 0;
    named_barrier(1, NT);
    if (!last) return;
    __threadfence();
    const int C = e.n_cols, R = C >> 1;
    double *red = reinterpret_cast<double *>(scratch);            // [NT][4]
    double *tot = red + NT * 4;                                   // [128][4]
    for (int slot0 = 0; slot0 < R; slot0 += 128) {
        const int cw = R - slot0 < 128 ? R - slot0 : 128;         // even
        reduce_records<NT>(e.part, (int)gridDim.x, C, slot0, cw, red, tot, etid);
        for (int lc = etid; lc < cw * 2; lc += NT) {              // one thread per channel of this slot range
            const int k = lc >> 2, j = lc & 3;                    // local quad, lane within it
            const int ch = (slot0 >> 1) * 4 + lc;
            const double sum = tot[(2 * k) * 4 + j], sum2 = tot[(2 * k + 1) * 4 + j];
            if (e.mode == EPI_BNBWD) {
                e.dbeta[ch] = (float)sum; e.dgamma[ch] = (float)sum2;
                const double gr = (double)e.bn.gamma[ch] * (double)e.bn.rstd[ch];
                e.coef[ch] = (float)gr; e.coef[C + ch] = (float)(gr * sum * e.inv_count); e.coef[2 * C + ch] = (float)(gr * sum2 * e.inv_count);
            } else {
                float m, r;
                moments_of(sum, sum2, e.inv_count, e.eps, m, r);
                e.mean[ch] = m; e.rstd[ch] = r;
            }
        }
        named_barrier(1, NT);
    }
    if (etid == 0) *e.counter = 0u;
}

}  // namespace tc
