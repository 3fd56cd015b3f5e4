// BN -> ReLU -> conv as ONE kernel for layers with at most 64 input channels (stride 1, k = 1 or 3):
// the layers whose cost is memory traffic, not arithmetic (Eq. 2: c_k(x) = Conv_kxk(ReLU(BN(x)))).
//
// All global traffic of a tile moves through TMA, asynchronously and (where shared memory allows)
// one tile ahead: the raw input tile WITH its halo (a 4-D box; what lies outside the image arrives
// as zeros), the tile the epilogue needs besides the accumulator (the coupling partner, or the BN
// input of a data gradient), and the finished output tile (a TMA store).  The threads only work
// between shared memory, registers and tensor memory:
//   - build: scale*x + shift, ReLU, bf16 rounding (pixels outside the image become zero: the
//     convolution pads the activated tensor, not the raw one), written in the swizzled K-major
//     layout tcgen05.mma reads -- k copies, one per horizontal tap offset, so that every tap's
//     operand is a contiguous run of 128 pixel rows of one copy: rows are ordered (image row,
//     image, column), a vertical tap offset is then a whole number of 8-row groups;
//   - one thread issues the MMAs (weights resident in shared memory, fp32 accumulator in tensor memory);
//   - epilogue: accumulator row + partner -> output tile in shared memory (Section 3.1 coupling on
//     the float or fixed-point state), then per-channel sums over the tile (batch statistics of
//     the stored result, or the two sums of the BN+ReLU backward), reduced over the grid by the
//     CTA that finishes last (conv_epilogue.cuh).
// The same kernel computes data gradients: its input is then the bf16 upstream gradient, taken as
// it is, and the weights are the mirrored, transposed pack.
// 128 threads per CTA, persistent over tiles blockIdx.x, blockIdx.x + gridDim.x, ...; small shapes
// run two CTAs per SM.  Every mbarrier wait is bounded and done by one thread; the rest block on
// a CTA barrier behind it.
#include "common.cuh"
#include "tc_ptx.cuh"
#include "conv_epilogue.cuh"
#include <cuda.h>
#include <string.h>

using namespace tc;

namespace {

constexpr int kFThreads = 256;     // warps 0-3 also drain the accumulator (warp w owns tensor-memory lanes 32w..32w+31)

struct FusedParams {
    int k;                 // 1 or 3
    int KC;                // padded input channels: 16, 32 or 64 (one K chunk)
    int cin;               // valid input channels (multiple of 8)
    int BN;                // output channels per N tile (multiple of 16, <= 128)
    int NB;                // buffers for the input and partner tiles (2: the next tile is loaded while this one is worked on)
    int copy_bytes;        // one shifted copy: (BH + k - 1) * BIMG * Wp rows of KC bf16, rounded up to 1024
    int wtile_bytes;       // one tap of the weights: BN rows of KC bf16, rounded up to 1024
    int a_bytes;           // operand region (k copies)
    int raw_bytes;         // one raw input tile with halo, rounded up to 128
    int aux_bytes;         // one partner / output tile: BN / GW column groups of group_bytes
    int GW;                // floats per row of a column group (16 or 32): rows of 64 / 128 bytes, stored with the matching TMA swizzle
    int group_bytes;       // tile pixels x GW floats, rounded up to 1024
    TileGeom g;            // hw_order = 1
    int in_mode;           // 0: float / fixed-point tensor through BN + ReLU; 1: bf16 tensor as it is
    float in_q;            // in_mode 0: fixed-point step of the input (0: float)
    BnRef bn;              // in_mode 0
    bf16 *a_out;           // in_mode 0, optional: the activated tensor [P, cin] written out (operand of the weight gradient)
    EpiArgs epi;           // out / partner / t are addressed through the tensor maps; their .q gives the format
    int *status;
    unsigned long long *stamp;    // timeline slot of this launch (nullptr: off)
};

struct __align__(16) FusedShared {
    uint64_t raw_full[2], aux_full[2], mma_done, w_full;
    uint32_t tmem_base, failed;
    RowMap rows;
    int srow[128];                   // accumulator row -> pixel index inside the partner / output tile (box order), -1: padding
    __align__(16) float sc[64];      // BN scale and shift per input channel
    __align__(16) float sf[64];
    __align__(16) uint4 dummy;             // where operand stores that have no destination go
    __align__(16) uint64_t desc[2 * 36];   // (operand, weight) descriptor of every MMA of a tile: they do not depend on the tile
};

// two floats -> ReLU -> bf16x2 (round to nearest even), one instruction
__device__ __forceinline__ uint32_t relu_pack2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Per pixel of the raw tile (in the order TMA delivers it: image, row, column), decoded once per CTA:
//   r01, r2 : row of the pixel in operand copy 0 / 1 (low / high half of r01) and copy 2 (low half of r2f),
//             0xffff where that copy does not hold it
//   r2f     : bits 16-23 halo row, 24-31 image in tile
//   flags   : bit 0: inside the tile proper (not halo); bit 1: column inside the image; bits 8-15: halo column
struct __align__(16) ItemRef { uint32_t r01, r2f, spare, flags; };

// a / b for 0 <= a < 65536 with inv_b = 1.f / b: exact, without the integer-division sequence
__device__ __forceinline__ int small_div(int a, float inv_b) { return __float2int_rz(((float)a + 0.5f) * inv_b); }

__device__ __forceinline__ void build_table(const FusedParams &p, ItemRef *tab, int npix) {
    const int pad = p.k >> 1;
    const int WH = p.g.W + 2 * pad, HR = p.g.BH + 2 * pad;
    const float inv_wh = 1.f / (float)WH, inv_hr = 1.f / (float)HR;
    for (int px = threadIdx.x; px < npix; px += kFThreads) {
        const int rest = small_div(px, inv_wh), xh = px - rest * WH;
        const int img = small_div(rest, inv_hr), r = rest - img * HR;
        const int rowbase = (r * p.g.BIMG + img) * p.g.Wp;
        const bool xin = xh >= pad && xh < pad + p.g.W;
        const bool interior = xin && r >= pad && r < pad + p.g.BH;
        uint32_t d[3];
#pragma unroll
        for (int s = 0; s < 3; s++) {            // halo column xh is column xh - s of the copy for horizontal tap offset s
            const int x = xh - s;
            d[s] = (s < p.k && x >= 0 && x < p.g.W) ? (uint32_t)(rowbase + x) : 0xffffu;
        }
        ItemRef e;
        e.r01 = d[0] | (d[1] << 16);
        e.r2f = d[2] | ((uint32_t)r << 16) | ((uint32_t)img << 24);
        e.spare = 0;
        e.flags = (interior ? 1u : 0u) | (xin ? 2u : 0u) | ((uint32_t)xh << 8);
        tab[px] = e;
    }
}

// raw tile (shared memory) -> operand copies (shared memory), NJ items per thread in flight (two
// where a tile has at most two items per thread: slots without an item would still cost their instructions).
// This thread's channel chunk ck is fixed: the thread count is a multiple of the chunks per pixel.
// IN_MODE 0: float input through BN + ReLU; 2: fixed-point input through BN + ReLU; 1: bf16 input as it is.
// Written without branches in the per-item work (invalid items compute on the zeros TMA delivered and are
// masked, stores that do not exist go to a dummy slot), so that the four items of a batch interleave.
template <int IN_MODE, int NJ>
__device__ __forceinline__ void build_tile(const FusedParams &p, FusedShared *sh, const ItemRef *tab, int items, int cshift, int ck,
                                           const uint8_t *raw, uint8_t *A, int n0, int h0) {
    const int pad = p.k >> 1;
    // 16-byte slot of chunk ck in row `row` of a copy: the chunk index is XORed with row bits as the TMA swizzle does
    const int swz_sh = 3 - cshift;
    const uint32_t swz_mask = (1u << cshift) - 1u;
    const bool ck_valid = ck < (p.cin >> 3);
    const uint32_t raw_px16 = (uint32_t)(p.cin * (IN_MODE == 1 ? 2 : 4)) >> 4, raw_ck16 = (uint32_t)(ck * (IN_MODE == 1 ? 1 : 2));
    // scale and shift of this thread's eight channels; a fixed-point input folds its step into the scale (a power of two: exact)
    float sc[8], sf[8];
    if (IN_MODE != 1) {
#pragma unroll
        for (int e = 0; e < 8; e++) { sc[e] = sh->sc[ck * 8 + e] * (IN_MODE == 2 ? p.in_q : 1.f); sf[e] = sh->sf[ck * 8 + e]; }
    }
    const uint32_t dummy = (uint32_t)(reinterpret_cast<uint8_t *>(&sh->dummy) - A);     // byte offset of the dummy slot relative to A
#pragma unroll 1
    for (int base = threadIdx.x; base < items; base += NJ * kFThreads) {
        ItemRef ref[NJ];
        uint4 v[NJ];
        bool ok[NJ];
#pragma unroll
        for (int j = 0; j < NJ; j++) {
            const int it = base + j * kFThreads;
            const bool exists = it < items;
            const uint32_t px = (uint32_t)(exists ? it : items - 1) >> cshift;
            ref[j] = tab[px];
            const int r = (ref[j].r2f >> 16) & 0xff, img = ref[j].r2f >> 24;
            ok[j] = exists && ck_valid && (ref[j].flags & 2u) && (unsigned)(h0 - pad + r) < (unsigned)p.g.H && n0 + img < p.g.N;
            if (!exists) { ref[j].r01 = 0xffffffffu; ref[j].r2f |= 0xffffu; }
            const uint4 *src = reinterpret_cast<const uint4 *>(raw) + (px * raw_px16 + raw_ck16);
            const uint4 lo = src[0];
            if (IN_MODE == 1) {
                v[j] = lo;
            } else {
                const uint4 hi = src[1];
                float x[8];
                if (IN_MODE == 0) {
                    x[0] = __uint_as_float(lo.x); x[1] = __uint_as_float(lo.y); x[2] = __uint_as_float(lo.z); x[3] = __uint_as_float(lo.w);
                    x[4] = __uint_as_float(hi.x); x[5] = __uint_as_float(hi.y); x[6] = __uint_as_float(hi.z); x[7] = __uint_as_float(hi.w);
                } else {
                    x[0] = __int2float_rn((int)lo.x); x[1] = __int2float_rn((int)lo.y); x[2] = __int2float_rn((int)lo.z); x[3] = __int2float_rn((int)lo.w);
                    x[4] = __int2float_rn((int)hi.x); x[5] = __int2float_rn((int)hi.y); x[6] = __int2float_rn((int)hi.z); x[7] = __int2float_rn((int)hi.w);
                }
#pragma unroll
                for (int e = 0; e < 8; e++) x[e] = fmaf(sc[e], x[e], sf[e]);
                v[j] = make_uint4(relu_pack2(x[0], x[1]), relu_pack2(x[2], x[3]), relu_pack2(x[4], x[5]), relu_pack2(x[6], x[7]));
            }
            const uint32_t keep = ok[j] ? 0xffffffffu : 0u;       // outside the image: zero, whatever BN makes of the zeros delivered
            v[j].x &= keep; v[j].y &= keep; v[j].z &= keep; v[j].w &= keep;
            const uint32_t r0 = ref[j].r01 & 0xffffu, r1 = ref[j].r01 >> 16, r2 = ref[j].r2f & 0xffffu;
            const uint32_t o0 = ((r0 << cshift) + ((uint32_t)ck ^ ((r0 >> swz_sh) & swz_mask))) << 4;
            const uint32_t o1 = ((r1 << cshift) + ((uint32_t)ck ^ ((r1 >> swz_sh) & swz_mask))) << 4;
            const uint32_t o2 = ((r2 << cshift) + ((uint32_t)ck ^ ((r2 >> swz_sh) & swz_mask))) << 4;
            *reinterpret_cast<uint4 *>(A + (r0 != 0xffffu ? o0 : dummy)) = v[j];
            *reinterpret_cast<uint4 *>(A + (r1 != 0xffffu ? p.copy_bytes + o1 : dummy)) = v[j];
            *reinterpret_cast<uint4 *>(A + (r2 != 0xffffu ? 2 * p.copy_bytes + o2 : dummy)) = v[j];
        }
        if (IN_MODE != 1 && p.a_out) {
#pragma unroll
            for (int j = 0; j < NJ; j++)
                if (ok[j] && (ref[j].flags & 1u)) {
                    const int r = (ref[j].r2f >> 16) & 0xff, img = ref[j].r2f >> 24, xh = (ref[j].flags >> 8) & 0xff;
                    const size_t gp = ((size_t)(n0 + img) * p.g.H + (h0 - pad + r)) * p.g.W + (xh - pad);
                    *reinterpret_cast<uint4 *>(p.a_out + gp * p.cin + ck * 8) = v[j];
                }
        }
    }
}

// Epilogue pass A for one thread (= one accumulator row, alternate groups of 8 columns): accumulator
// (+ partner tile) -> output tile in shared memory.  KIND: 0 plain float, 1 plain onto the fixed-point
// grid, 2 / 3 float coupling + / -, 4 / 5 fixed-point coupling + / -.  One instantiation per kind, so
// that the loop body has no branches.
template <int KIND>
__device__ __forceinline__ void pass_a(const FusedParams &p, uint32_t tm, int c0, int sr, const uint8_t *aux, uint8_t *outb,
                                       float out_s, int row_b) {
    const int swz = p.GW == 32 ? (sr & 7) : ((sr >> 1) & 3);
#pragma unroll 1
    for (int c = c0; c < p.BN; c += 16) {
        float v[8];
        tmem_ld8(tm + (uint32_t)c, v);
        if (sr < 0) continue;
        const int gbase = (c / p.GW) * p.group_bytes + sr * row_b, j0 = (c % p.GW) >> 2;
#pragma unroll
        for (int j = 0; j < 2; j++) {
            const int off = gbase + (((j0 + j) ^ swz) << 4);
            float4 r = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            if (KIND == 2 || KIND == 3) {
                const float4 pr = *reinterpret_cast<const float4 *>(aux + off);
                if (KIND == 2) { r.x = pr.x + r.x; r.y = pr.y + r.y; r.z = pr.z + r.z; r.w = pr.w + r.w; }
                else { r.x = pr.x - r.x; r.y = pr.y - r.y; r.z = pr.z - r.z; r.w = pr.w - r.w; }
            } else if (KIND != 0) {
                int4 iv = make_int4(__float2int_rn(r.x * out_s), __float2int_rn(r.y * out_s), __float2int_rn(r.z * out_s), __float2int_rn(r.w * out_s));
                if (KIND >= 4) {
                    const int4 pi = *reinterpret_cast<const int4 *>(aux + off);
                    if (KIND == 4) { iv.x = pi.x + iv.x; iv.y = pi.y + iv.y; iv.z = pi.z + iv.z; iv.w = pi.w + iv.w; }
                    else { iv.x = pi.x - iv.x; iv.y = pi.y - iv.y; iv.z = pi.z - iv.z; iv.w = pi.w - iv.w; }
                }
                r = make_float4(__int_as_float(iv.x), __int_as_float(iv.y), __int_as_float(iv.z), __int_as_float(iv.w));
            }
            *reinterpret_cast<float4 *>(outb + off) = r;
        }
    }
}

// Epilogue pass B for one thread (= one channel quad, every rpp-th pixel): running per-channel sums over
// the valid pixels of the output tile.  KIND 0 / 1: sums and second sums of the stored values (float /
// fixed point); 2 / 3: the two sums of the BN+ReLU backward with a float / fixed-point BN input tile.
// Rows are added in a fixed order.
template <int KIND>
__device__ __forceinline__ void pass_b(const FusedParams &p, const uint8_t *ob, const uint8_t *aux, int jq, int r0, int rpp, int valid_px,
                                       int row_b, float q, float4 sc4, float4 sh4, float4 mu4, float4 rs4, float (&acc)[8]) {
#pragma unroll 4
    for (int pl = r0; pl < valid_px; pl += rpp) {
        const int off = pl * row_b + ((jq ^ (p.GW == 32 ? (pl & 7) : ((pl >> 1) & 3))) << 4);
        float4 v = *reinterpret_cast<const float4 *>(ob + off);
        if (KIND >= 2) {
            float4 tt = *reinterpret_cast<const float4 *>(aux + off);
            if (KIND == 3) tt = make_float4(__int2float_rn(__float_as_int(tt.x)) * q, __int2float_rn(__float_as_int(tt.y)) * q,
                                            __int2float_rn(__float_as_int(tt.z)) * q, __int2float_rn(__float_as_int(tt.w)) * q);
            const float dx = fmaf(sc4.x, tt.x, sh4.x) > 0.f ? v.x : 0.f, dy = fmaf(sc4.y, tt.y, sh4.y) > 0.f ? v.y : 0.f;
            const float dz = fmaf(sc4.z, tt.z, sh4.z) > 0.f ? v.z : 0.f, dw = fmaf(sc4.w, tt.w, sh4.w) > 0.f ? v.w : 0.f;
            acc[0] += dx; acc[1] += dy; acc[2] += dz; acc[3] += dw;
            acc[4] += dx * ((tt.x - mu4.x) * rs4.x); acc[5] += dy * ((tt.y - mu4.y) * rs4.y);
            acc[6] += dz * ((tt.z - mu4.z) * rs4.z); acc[7] += dw * ((tt.w - mu4.w) * rs4.w);
        } else {
            if (KIND == 1) v = make_float4(__int2float_rn(__float_as_int(v.x)) * q, __int2float_rn(__float_as_int(v.y)) * q,
                                           __int2float_rn(__float_as_int(v.z)) * q, __int2float_rn(__float_as_int(v.w)) * q);
            acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
            acc[4] += v.x * v.x; acc[5] += v.y * v.y; acc[6] += v.z * v.z; acc[7] += v.w * v.w;
        }
    }
}

// One tile's place in the tensor.  Tiles are stepped by the grid size without divisions.
struct TilePos { int t, n0, h0, hidx; };
struct TileStep { int gq, gr; };     // grid size = gq whole images + gr row tiles (BIMG == 1)
__device__ __forceinline__ void tile_first(const TileGeom &g, int t, TilePos &tp) {
    tp.t = t;
    if (g.BIMG > 1) { tp.n0 = t * g.BIMG; tp.h0 = 0; tp.hidx = 0; }
    else { tp.n0 = t / g.tiles_per_img; tp.hidx = t - tp.n0 * g.tiles_per_img; tp.h0 = tp.hidx * g.BH; }
}
__device__ __forceinline__ void tile_next(const TileGeom &g, const TileStep &st, int G, TilePos &tp) {
    tp.t += G;
    if (g.BIMG > 1) { tp.n0 += G * g.BIMG; return; }
    tp.n0 += st.gq; tp.hidx += st.gr;
    if (tp.hidx >= g.tiles_per_img) { tp.hidx -= g.tiles_per_img; tp.n0++; }
    tp.h0 = tp.hidx * g.BH;
}

__global__ void __launch_bounds__(kFThreads, 2)
conv_fused_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_in,
                  const __grid_constant__ CUtensorMap map_aux, const __grid_constant__ CUtensorMap map_out, const FusedParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *abuf = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int taps = p.k * p.k;
    uint8_t *wres = abuf + p.a_bytes;
    uint8_t *rawb = wres + taps * p.wtile_bytes;
    uint8_t *auxb = rawb + p.NB * p.raw_bytes;
    uint8_t *outb = auxb + p.NB * p.aux_bytes;
    FusedShared *sh = (FusedShared *)(outb + p.aux_bytes);
    ItemRef *tab = (ItemRef *)(sh + 1);

    const int warp = threadIdx.x >> 5;
    const int etid = threadIdx.x & 127;                 // warps 0-3: accumulator row; all warps: index for the reductions
    const int cshift = p.KC == 64 ? 3 : (p.KC == 32 ? 2 : 1);     // 16-byte chunks per pixel = KC / 8
    const int pad = p.k >> 1;
    const int npix = (p.g.BH + 2 * pad) * p.g.BIMG * (p.g.W + 2 * pad);
    const int items = npix << cshift;
    const int tile_px = p.g.BH * p.g.BIMG * p.g.W;      // pixels of a partner / output tile
    // one accumulator: splitting the taps over several (summed in the epilogue) was measured slower
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < p.BN) tmem_cols <<= 1;
    const int col0 = blockIdx.y * p.BN;
    const int row_bytes = p.KC * 2;
    const EpiArgs &e = p.epi;
    const bool need_aux = e.mode != EPI_PLAIN;
    const uint32_t raw_tx = (uint32_t)(npix * p.cin * (p.in_mode == 0 ? 4 : 2));
    const uint32_t aux_tx = (uint32_t)(tile_px * p.BN * 4);

    const int G = (int)gridDim.x, NT = p.g.n_px_tiles;
    TileStep step;
    step.gq = p.g.BIMG > 1 ? 0 : G / p.g.tiles_per_img;
    step.gr = p.g.BIMG > 1 ? 0 : G - step.gq * p.g.tiles_per_img;
    auto load_raw = [&](const TilePos &tp, int b) {     // thread 0
        mbar_expect_tx(&sh->raw_full[b], raw_tx);
        tma_load_4d(rawb + b * p.raw_bytes, &map_in, &sh->raw_full[b], 0, -pad, tp.h0 - pad, tp.n0);
    };
    auto load_aux = [&](const TilePos &tp, int b) {
        mbar_expect_tx(&sh->aux_full[b], aux_tx);
        for (int g = 0; g < p.BN / p.GW; g++)
            tma_load_4d(auxb + b * p.aux_bytes + g * p.group_bytes, &map_aux, &sh->aux_full[b], col0 + g * p.GW, 0, tp.h0, tp.n0);
    };
    TilePos cur, nx1, nx2;             // this tile, the next one and the one after
    tile_first(p.g, blockIdx.x, cur);
    nx1 = cur; tile_next(p.g, step, G, nx1);
    nx2 = nx1; tile_next(p.g, step, G, nx2);
    // inside a column group pixel r has a row of 128 (64) bytes whose 16-byte chunks are XORed with address bits 7..
    // as the TMA swizzle does, so that a thread per row touches all banks
    const int row_b = p.GW * 4;

    if (threadIdx.x == 0) {
        for (int b = 0; b < 2; b++) { mbar_init(&sh->raw_full[b], 1); mbar_init(&sh->aux_full[b], 1); }
        mbar_init(&sh->mma_done, 1);
        mbar_init(&sh->w_full, 1);
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_w); tma_prefetch_desc(&map_in); tma_prefetch_desc(&map_out);
        if (need_aux) tma_prefetch_desc(&map_aux);
        // the first loads fly while the CTA builds its index tables
        pdl_enter();
        mbar_expect_tx(&sh->w_full, (uint32_t)(taps * p.BN * p.KC * 2));
        for (int tap = 0; tap < taps; tap++) tma_load_2d(wres + tap * p.wtile_bytes, &map_w, &sh->w_full, tap * p.KC, col0);
        if (cur.t < NT) {
            load_raw(cur, 0);
            if (need_aux) load_aux(cur, 0);
            if (p.NB == 2 && nx1.t < NT) load_raw(nx1, 1);
        }
    }
    if (warp == 0) tmem_alloc(&sh->tmem_base, tmem_cols);
    build_table(p, tab, npix);
    if (threadIdx.x < 128) {
        // accumulator row (image row, image, column) -> pixel of the (image, row, column) ordered tile
        const int w = etid % p.g.Wp, img = (etid / p.g.Wp) % p.g.BIMG, h = etid / (p.g.BIMG * p.g.Wp);
        sh->srow[etid] = (w < p.g.W && h < p.g.BH) ? (img * p.g.BH + h) * p.g.W + w : -1;
    }
    // the tables above are independent of what earlier kernels wrote; everything below is not
    pdl_enter();
    stamp_begin(p.stamp);
    if (p.in_mode == 0 && p.bn.part) {
        // the statistics of the input are still per-CTA records of the kernel before: add them here (every CTA
        // the same way, while its first tile is on the way); the first CTA stores mean and rstd for later readers
        double *red = reinterpret_cast<double *>(abuf), *tot = red + kFThreads * 4;
        reduce_records<kFThreads>(p.bn.part, p.bn.parts, p.cin, 0, p.cin >> 1, red, tot, (int)threadIdx.x);
        if (threadIdx.x < 64) {
            const int c = threadIdx.x;
            float sc = 0.f, sf = 0.f;
            if (c < p.cin) {
                float mean, rstd;
                moments_of(tot[(2 * (c >> 2)) * 4 + (c & 3)], tot[(2 * (c >> 2) + 1) * 4 + (c & 3)], p.bn.inv_count, p.bn.eps, mean, rstd);
                if (blockIdx.x == 0 && blockIdx.y == 0) { const_cast<float *>(p.bn.mean)[c] = mean; const_cast<float *>(p.bn.rstd)[c] = rstd; }
                bn_sc_sh(p.bn.gamma[c], p.bn.beta[c], mean, rstd, sc, sf);
            }
            sh->sc[c] = sc; sh->sf[c] = sf;
        }
    } else if (threadIdx.x >= 128 && threadIdx.x < 192) {
        const int c = threadIdx.x - 128;
        float sc = 0.f, sf = 0.f;
        if (p.in_mode == 0 && c < p.cin) bn_sc_sh(p.bn.gamma[c], p.bn.beta[c], p.bn.mean[c], p.bn.rstd[c], sc, sf);
        sh->sc[c] = sc; sh->sf[c] = sf;
    }
    if (threadIdx.x == 224) {
        // descriptors differ between taps and K steps only in their start-address field (16-byte units)
        const uint32_t row_group = (uint32_t)(p.g.BIMG * p.g.Wp * row_bytes);     // one image row of the tile, in bytes
        const uint64_t a_desc = smem_desc(smem_u32(abuf), row_bytes), w_desc = smem_desc(smem_u32(wres), row_bytes);
        int i = 0;
        for (int kh = 0; kh < p.k; kh++)
            for (int kw = 0; kw < p.k; kw++)
                for (int kk = 0; kk < (p.KC >> 4); kk++, i++) {
                    sh->desc[2 * i] = a_desc + (uint64_t)(((kw * p.copy_bytes + kh * row_group) >> 4) + kk * 2);
                    sh->desc[2 * i + 1] = w_desc + (uint64_t)((((kh * p.k + kw) * p.wtile_bytes) >> 4) + kk * 2);
                }
    }
    const int ck = threadIdx.x & ((1 << cshift) - 1);      // this thread's channel chunk
    // reductions: this thread's channel quad and its running sums
    const int QW = p.BN >> 2, rpp = kFThreads / QW;
    const int quad = (int)threadIdx.x % QW, r0 = (int)threadIdx.x / QW;
    const bool reducer = e.part && r0 < rpp && col0 + quad * 4 < e.n_cols;
    float4 sc4 = make_float4(0, 0, 0, 0), sh4 = sc4, mu4 = sc4, rs4 = sc4;
    if (reducer && e.mode == EPI_BNBWD) bn_coef4(e.bn, col0 + quad * 4, sc4, sh4, mu4, rs4);
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f, q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = sh->tmem_base;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const float out_q = e.out.q, out_s = out_q != 0.f ? 1.f / out_q : 0.f;
    const float t_q = e.t.q;
    bool ok = true;
    int ti = 0;
#pragma unroll 1
    for (; cur.t < NT; ti++) {
        const int b = ti % p.NB; const uint32_t u = ti / p.NB;
        const int n0 = cur.n0, h0 = cur.h0;
        // with two buffers the loads of the tiles ahead are issued while this tile's MMAs run (below)
        if (threadIdx.x == 0) ok = mbar_wait(&sh->raw_full[b], u & 1);
        ok = __syncthreads_and(ok);
        if (!ok) break;
        // ---- build the operand
        if (items <= 2 * kFThreads) {
            if (p.in_mode == 1) build_tile<1, 2>(p, sh, tab, items, cshift, ck, rawb + b * p.raw_bytes, abuf, n0, h0);
            else if (p.in_q == 0.f) build_tile<0, 2>(p, sh, tab, items, cshift, ck, rawb + b * p.raw_bytes, abuf, n0, h0);
            else build_tile<2, 2>(p, sh, tab, items, cshift, ck, rawb + b * p.raw_bytes, abuf, n0, h0);
        } else {
            if (p.in_mode == 1) build_tile<1, 4>(p, sh, tab, items, cshift, ck, rawb + b * p.raw_bytes, abuf, n0, h0);
            else if (p.in_q == 0.f) build_tile<0, 4>(p, sh, tab, items, cshift, ck, rawb + b * p.raw_bytes, abuf, n0, h0);
            else build_tile<2, 4>(p, sh, tab, items, cshift, ck, rawb + b * p.raw_bytes, abuf, n0, h0);
        }
        fence_proxy_async();
        __syncthreads();
        if (threadIdx.x == 0) {
            if (p.NB == 1 && nx1.t < NT) load_raw(nx1, 0);        // the raw buffer is free again
            if (ti == 0 && !mbar_wait(&sh->w_full, 0)) ok = false;
            tc_fence_after();
            const uint32_t idesc = instr_desc(p.BN);
            const int n_mma = taps * (p.KC >> 4);
            const ulonglong2 *dsc = reinterpret_cast<const ulonglong2 *>(sh->desc);
#pragma unroll 4
            for (int i = 0; i < n_mma; i++) {
                const ulonglong2 d = dsc[i];
                mma_bf16(tmem_d, d.x, d.y, idesc, i ? 1u : 0u);
            }
            mma_commit(&sh->mma_done);
            tma_store_wait_read();                       // the previous tile's store has read the output buffer
            ok = ok && mbar_wait(&sh->mma_done, ti & 1) && (!need_aux || mbar_wait(&sh->aux_full[b], u & 1));
        }
        else if (threadIdx.x == 32 && p.NB == 2) {
            // meanwhile another thread issues the loads of the tiles ahead: this tile's raw buffer has been consumed,
            // and the other partner buffer was last read by the epilogue before
            if (nx2.t < NT) load_raw(nx2, b);
            if (need_aux && nx1.t < NT) load_aux(nx1, b ^ 1);
        }
        ok = __syncthreads_and(ok);
        if (!ok) break;
        tc_fence_after();
        // ---- epilogue, pass A: accumulator row (+ partner) -> output tile in shared memory
        {
            // all eight warps: warp w and w + 4 share tensor-memory lanes 32(w%4).. and take alternate groups of 8 columns
            const int sr = sh->srow[etid];
            const uint8_t *aux = auxb + b * p.aux_bytes;
            const uint32_t tm = tmem_d + lane_base;
            const int c0 = (warp >> 2) * 8;
            if (e.mode != EPI_COUPLE) {
                if (out_q == 0.f) pass_a<0>(p, tm, c0, sr, aux, outb, out_s, row_b);
                else pass_a<1>(p, tm, c0, sr, aux, outb, out_s, row_b);
            } else if (out_q == 0.f) {
                if (e.sign > 0) pass_a<2>(p, tm, c0, sr, aux, outb, out_s, row_b); else pass_a<3>(p, tm, c0, sr, aux, outb, out_s, row_b);
            } else {
                if (e.sign > 0) pass_a<4>(p, tm, c0, sr, aux, outb, out_s, row_b); else pass_a<5>(p, tm, c0, sr, aux, outb, out_s, row_b);
            }
        }
        fence_proxy_async();
        tc_fence_before();       // the next tile's MMAs overwrite the accumulator
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int g = 0; g < p.BN / p.GW; g++) tma_store_4d(&map_out, outb + g * p.group_bytes, col0 + g * p.GW, 0, h0, n0);
            tma_store_commit();
        }
        // ---- pass B: per-channel sums over the valid pixels of the tile (a prefix in the tile's pixel order)
        if (reducer) {
            int valid_px = p.g.BIMG > 1 ? (p.g.N - n0 < p.g.BIMG ? p.g.N - n0 : p.g.BIMG) * p.g.BH * p.g.W
                                        : (p.g.H - h0 < p.g.BH ? p.g.H - h0 : p.g.BH) * p.g.W;
            const int qg = p.GW >> 2;                      // quads per column group
            const uint32_t gb = (uint32_t)((quad / qg) * p.group_bytes);
            const int jq = quad % qg;
            const uint8_t *aux = auxb + b * p.aux_bytes + gb;
            const uint8_t *ob = outb + gb;
            float acc[8] = {s0, s1, s2, s3, q0, q1, q2, q3};
            if (e.mode == EPI_BNBWD) {
                if (t_q == 0.f) pass_b<2>(p, ob, aux, jq, r0, rpp, valid_px, row_b, 0.f, sc4, sh4, mu4, rs4, acc);
                else pass_b<3>(p, ob, aux, jq, r0, rpp, valid_px, row_b, t_q, sc4, sh4, mu4, rs4, acc);
            } else if (out_q == 0.f) pass_b<0>(p, ob, aux, jq, r0, rpp, valid_px, row_b, 0.f, sc4, sh4, mu4, rs4, acc);
            else pass_b<1>(p, ob, aux, jq, r0, rpp, valid_px, row_b, out_q, sc4, sh4, mu4, rs4, acc);
            s0 = acc[0]; s1 = acc[1]; s2 = acc[2]; s3 = acc[3]; q0 = acc[4]; q1 = acc[5]; q2 = acc[6]; q3 = acc[7];
        }
        if (p.NB == 1) {
            __syncthreads();     // the partner buffer is free
            if (threadIdx.x == 0 && need_aux && nx1.t < NT) load_aux(nx1, 0);
        }
        cur = nx1; nx1 = nx2;
        tile_next(p.g, step, G, nx2);
    }
    if (threadIdx.x == 0) tma_store_wait_all();
    if (ok && e.part) {
        // per-CTA record: the threads that share a channel quad are added in order
        float *scratch = reinterpret_cast<float *>(abuf);
        float *mysl = scratch + threadIdx.x * 8;
        mysl[0] = s0; mysl[1] = s1; mysl[2] = s2; mysl[3] = s3; mysl[4] = q0; mysl[5] = q1; mysl[6] = q2; mysl[7] = q3;
        __syncthreads();
        if (reducer && r0 == 0) {
            float r[8];
#pragma unroll
            for (int j = 0; j < 8; j++) r[j] = scratch[quad * 8 + j];
            for (int y = 1; y < rpp; y++)
#pragma unroll
                for (int j = 0; j < 8; j++) r[j] += scratch[(y * QW + quad) * 8 + j];
            float *mine = e.part + (size_t)blockIdx.x * 2 * e.n_cols + 2 * (col0 + quad * 4);
            *reinterpret_cast<float4 *>(mine) = make_float4(r[0], r[1], r[2], r[3]);
            *reinterpret_cast<float4 *>(mine + 4) = make_float4(r[4], r[5], r[6], r[7]);
        }
        __syncthreads();
        if (e.counter) epilogue_publish<kFThreads>(e, scratch, (int)threadIdx.x);     // else the consumer adds the records
    }
    if (!ok && threadIdx.x == 0) atomicExch(&sh->failed, 1u);
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && sh->failed) atomicExch(p.status, (int)REVNET_E_TIMEOUT);
    stamp_end(p.stamp);
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_d, tmem_cols);
    }
}

int round_up(int x, int m) { return (x + m - 1) / m * m; }

// tiles of the fused kernel: accumulator rows run (image row, image, column) with the column pitch rounded up to 8
bool fused_tile_geom(Geom g, TileGeom &t) {
    t.N = g.N; t.H = g.H; t.W = g.W; t.hw_order = 1;
    t.Wp = round_up(g.W, 8);
    if (t.Wp > 128) return false;
    t.BH = 128 / t.Wp; if (t.BH > g.H) t.BH = g.H;
    t.BIMG = 1;
    if (t.BH == g.H) { t.BIMG = 128 / (g.H * t.Wp); if (t.BIMG > g.N) t.BIMG = g.N; if (t.BIMG < 1) t.BIMG = 1; }
    t.tiles_per_img = (g.H + t.BH - 1) / t.BH;
    t.n_px_tiles = t.BIMG > 1 ? (g.N + t.BIMG - 1) / t.BIMG : g.N * t.tiles_per_img;
    return true;
}

struct FusedShape { int KC, BN, n_tiles, NB, GW, group_bytes, copy_bytes, wtile_bytes, a_bytes, raw_bytes, aux_bytes, smem, occ; TileGeom g; };

bool fused_shape(Geom g, int cin, int cout, int k, int in_esize, int sm_count, FusedShape &s) {
    if ((k != 1 && k != 3) || cin % 8 || cout % 4 || cin < 8) return false;
    s.KC = round_up(cin, 16);
    if (s.KC != 16 && s.KC != 32 && s.KC != 64) return false;
    if (!fused_tile_geom(g, s.g)) return false;
    const int pad = k / 2;
    if (s.g.BH + 2 * pad > 255 || s.g.W + 2 * pad > 255 || s.g.BIMG > 255) return false;   // TMA box limits, fields of ItemRef
    const int cout_pad = round_up(cout, 16);
    s.BN = cout_pad <= 128 ? cout_pad : 128;
    // few pixel tiles (late stages): split the output channels so that more SMs take part
    while (s.BN % 32 == 0 && s.BN >= 32 && s.g.n_px_tiles * ((cout_pad + s.BN - 1) / s.BN) * 2 <= sm_count) s.BN /= 2;
    const int copy_rows = (s.g.BH + k - 1) * s.g.BIMG * s.g.Wp;
    s.copy_bytes = (copy_rows * s.KC * 2 + 1023) & ~1023;
    const int npix = (s.g.BH + 2 * pad) * s.g.BIMG * (s.g.W + 2 * pad);
    s.a_bytes = k * s.copy_bytes > 12288 ? k * s.copy_bytes : 12288;      // also scratch of the final reduction
    s.raw_bytes = (npix * cin * in_esize + 1023) & ~1023;
    for (;;) {
        s.n_tiles = (cout_pad + s.BN - 1) / s.BN;
        s.wtile_bytes = (s.BN * s.KC * 2 + 1023) & ~1023;
        s.GW = s.BN % 32 == 0 ? 32 : 16;
        s.group_bytes = (s.g.BH * s.g.BIMG * s.g.W * s.GW * 4 + 1023) & ~1023;
        s.aux_bytes = (s.BN / s.GW) * s.group_bytes;
        auto smem_of = [&](int NB) { return 1024 + s.a_bytes + k * k * s.wtile_bytes + NB * (s.raw_bytes + s.aux_bytes) + s.aux_bytes +
                                            (int)sizeof(FusedShared) + npix * 16 + 64; };
        const int two_per_sm = 113 * 1024;
        if (smem_of(2) <= two_per_sm) s.NB = 2;
        else if (smem_of(1) <= two_per_sm) s.NB = 1;
        else if (smem_of(2) <= 227 * 1024) s.NB = 2;
        else s.NB = 1;
        s.smem = smem_of(s.NB);
        if (s.smem <= 227 * 1024) { s.occ = s.smem <= two_per_sm ? 2 : 1; return true; }
        if (s.BN % 32 || s.BN < 32) return false;       // too large even single-buffered: narrower N tiles
        s.BN /= 2;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 4-D tensor map over an NHWC tensor of C channels: box = box_c channels x bw columns x bh rows x bimg images
bool encode_nhwc(EncodeTiledFn enc, CUtensorMap *map, CUtensorMapDataType dt, int esize, const void *base, Geom g, int C,
                 int box_c, int bw, int bh, int bimg, CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_NONE) {
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N};
    cuuint64_t strides[3] = {(cuuint64_t)C * esize, (cuuint64_t)g.W * C * esize, (cuuint64_t)g.H * g.W * C * esize};
    cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)bw, (cuuint32_t)bh, (cuuint32_t)bimg};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return enc(map, dt, 4, (void *)base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// in: [P, cin] float / fixed point (in_mode 0) or bf16 (in_mode 1); out, partner and the BN input of a
// data gradient must be plain (unsplit) tensors of cout channels
bool run_fused(Exec &ex, const char *what, int in_mode, const void *in, float in_q, BnRef bn, Geom g, int cin, int cout, int k,
               const float *Wsrc, const bf16 *prepacked, bool transposed, Pair out, Pair partner, int sign, EpiReq req, bf16 *a_out) {
    FusedShape s;
    if (out.c1 != 0 || (sign && partner.c1 != 0) || (req.bnbwd && req.bnbwd->t.c1 != 0)) return false;
    if (!fused_shape(g, cin, cout, k, in_mode == 0 ? 4 : 2, ex.ctx->sm_count, s)) return false;
    EncodeTiledFn enc = nullptr;
    if (!ex.dry) { enc = (EncodeTiledFn)tc_encoder(ex.ctx); if (!enc) return false; }
    const int taps = k * k, pad = k / 2;
    ex.flops += 2ull * g.P() * cout * cin * taps;
    int ctas = ex.ctx->sm_count * s.occ / s.n_tiles; if (ctas < 1) ctas = 1;
    if (ctas > s.g.n_px_tiles) ctas = s.g.n_px_tiles;
    size_t m = ex.ws.mark();
    const size_t pack_elems = tc_pack_elems(transposed ? cout : cin, transposed ? cin : cout, k, transposed);
    bf16 *wp = prepacked ? const_cast<bf16 *>(prepacked) : ex.ws.get<bf16>(pack_elems);
    const bool reduce = req.stats || req.bnbwd;
    // statistics whose owner has room for the records stay pending: the kernel that consumes them adds the records
    const bool defer = req.stats && !req.bnbwd && req.stats->part && (size_t)ctas * 2 * cout <= req.stats->part_cap;
    float *part = defer ? req.stats->part : (reduce ? ex.ws.get<float>((size_t)ctas * 2 * cout) : nullptr);
    if (req.stats) {
        req.stats->valid = true;
        req.stats->pending = defer; req.stats->parts = ctas; req.stats->inv_count = 1.0 / (double)g.P();
    }
    if (!ex.dry) {
        if (!prepacked) tc_pack_now(ex, Wsrc, wp, transposed ? cout : cin, transposed ? cin : cout, k, transposed);
        const int rows_pad = s.n_tiles * s.BN;
        CUtensorMap map_w, map_in, map_aux, map_out;
        const CUtensorMapSwizzle sw = s.KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (s.KC == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
        cuuint64_t dims[2] = {(cuuint64_t)taps * s.KC, (cuuint64_t)rows_pad};
        cuuint64_t strides[1] = {(cuuint64_t)taps * s.KC * 2};
        cuuint32_t box[2] = {(cuuint32_t)s.KC, (cuuint32_t)s.BN};
        cuuint32_t es[2] = {1, 1};
        bool maps_ok = enc(&map_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void *)wp, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        maps_ok = maps_ok && encode_nhwc(enc, &map_in, in_mode == 0 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                         in_mode == 0 ? 4 : 2, in, g, cin, cin, s.g.W + 2 * pad, s.g.BH + 2 * pad, s.g.BIMG);
        const CUtensorMapSwizzle gsw = s.GW == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
        maps_ok = maps_ok && encode_nhwc(enc, &map_out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, out.p0, g, cout, s.GW, s.g.W, s.g.BH, s.g.BIMG, gsw);
        const float *aux = req.bnbwd ? req.bnbwd->t.p0 : (sign ? partner.p0 : out.p0);
        maps_ok = maps_ok && encode_nhwc(enc, &map_aux, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, aux, g, cout, s.GW, s.g.W, s.g.BH, s.g.BIMG, gsw);
        if (!maps_ok) { ex.failed = true; ex.ctx->err = std::string(what) + ": tensor map rejected"; ex.ws.release(m); return true; }
        FusedParams p;
        memset(&p, 0, sizeof p);
        p.k = k; p.KC = s.KC; p.cin = cin; p.BN = s.BN; p.NB = s.NB; p.copy_bytes = s.copy_bytes; p.wtile_bytes = s.wtile_bytes;
        p.a_bytes = s.a_bytes; p.raw_bytes = s.raw_bytes; p.aux_bytes = s.aux_bytes; p.GW = s.GW; p.group_bytes = s.group_bytes; p.g = s.g;
        p.in_mode = in_mode; p.in_q = in_q; p.bn = bn; p.a_out = a_out; p.status = ex.ctx->dev_status; p.stamp = ex.stamp_slot();
        EpiArgs &e = p.epi;
        e.mode = req.bnbwd ? EPI_BNBWD : (sign ? EPI_COUPLE : EPI_PLAIN);
        e.out = out; e.partner = partner; e.sign = sign; e.n_cols = cout;
        e.part = part; e.counter = (reduce && !defer) ? ex.ctx->counter() : nullptr;
        e.inv_count = 1.0 / (double)g.P(); e.eps = ex.eps;
        if (req.stats) { e.mean = req.stats->mean; e.rstd = req.stats->rstd; }
        if (req.bnbwd) { e.t = req.bnbwd->t; e.bn = req.bnbwd->bn; e.dgamma = req.bnbwd->dgamma; e.dbeta = req.bnbwd->dbeta; e.coef = req.bnbwd->coef; }
        static OncePerDevice once;
        if (once.first(ex.ctx->device)) cudaFuncSetAttribute(conv_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        dim3 grid((unsigned)ctas, (unsigned)s.n_tiles);
        launch(ex, conv_fused_kernel, grid, kFThreads, s.smem, map_w, map_in, map_aux, map_out, p);
        const double bytes = (double)g.P() * cin * (in_mode == 0 ? 4 : 2) + (double)g.P() * cout * (sign || req.bnbwd ? 8 : 4) +
                             (double)cout * taps * cin * 2 + (a_out ? (double)g.P() * cin * 2 : 0.0);
        ex.check(what, bytes, 2.0 * g.P() * cout * cin * taps);
    }
    ex.ws.release(m);
    return true;
}

}  // namespace

// out = partner + sign * conv(ReLU(BN(t)));  a_out (optional): the activated tensor, for the weight gradient
bool conv_fprop_fused(Exec &ex, Pair t, BnRef bn, Geom gi, const Layer &L, Pair out, Pair partner, int sign, Moments *stats, bf16 *a_out) {
    if (L.stride != 1 || t.c1 != 0) return false;
    EpiReq req; req.stats = stats;
    return run_fused(ex, "conv_fprop_fused", 0, t.p0, t.q, bn, gi, L.cin, L.cout, L.k, L.W, L.Wp_fprop, false, out, partner, sign, req, a_out);
}

// da = conv^T(g) for a stride-1 layer, g bf16 [P, cout]
bool conv_dgrad_fused(Exec &ex, const void *g, Geom gi, const Layer &L, float *da, const BnBwdReq *bb) {
    if (L.stride != 1) return false;
    EpiReq req; req.bnbwd = bb;
    return run_fused(ex, "conv_dgrad_fused", 1, g, 0.f, BnRef{}, gi, L.cout, L.cin, L.k, L.W, L.Wp_dgrad, true, single(da, L.cin), Pair{}, 0, req, nullptr);
}
