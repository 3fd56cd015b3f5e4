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
// Roles inside a CTA: warp 0 issues TMA loads, warp 1 allocates tensor memory and issues the MMAs,
// the remaining warps drain the accumulator (tcgen05.ld), apply the coupling epilogue (out = partner
// +/- acc on the float or fixed-point state) and store: two groups of four warps (320 threads) where
// the epilogue's tiles move through TMA, one group (192 threads) in the staged form.
// Every mbarrier wait is bounded; on expiry the kernel records a status word and leaves.
#include "common.cuh"
#include "tc_ptx.cuh"
#include "conv_epilogue.cuh"
#include <cuda.h>
#include <string.h>
#include <stdlib.h>

using namespace tc;

namespace {

constexpr int kStages = 6;       // most operand stages of the convolution kernel
constexpr int kWgStages = 4;     // ... of the weight-gradient kernel
constexpr int kThreads = 192;      // TMA warp, MMA warp, four epilogue warps
constexpr int kThreadsTma = 320;   // epilogue through TMA: two groups of four epilogue warps

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
    int stages;      // operand ring depth (<= kStages)
    // epilogue through TMA (epi_tma): the output tile leaves, and the tile read besides the accumulator (coupling
    // partner, or BN input of a data gradient) arrives, as column groups of GW floats per pixel row
    int epi_tma;
    int GW;          // 32 or 16 floats: rows of 128 / 64 bytes, stored with the matching TMA swizzle
    int group_bytes; // one column group of a tile (128 pixel rows), a multiple of 1024
    int need_aux;
    int aux_slots;   // conv_tc2_kernel: slots of the partner ring (two interleaved rings, one per epilogue warp group)
    int split_o, split_x;   // channels in the first tensor of a channel-split output / partner (0: one tensor)
    // the taps this launch sums: offset of the operand box in rows / columns of the operand tensor, and the tap's
    // place in the weight pack.  A plain convolution lists all k*k taps; one parity class of a stride-2 data
    // gradient lists the one, two or four taps that reach its output pixels.
    // A launch with n_cls classes walks n_cls * n_px_tiles tiles: tile t belongs to class t / n_px_tiles (a plain
    // convolution has one class).  CTAs stride over that list, so every CTA gets its share of the short and long classes.
    int n_cls;
    int ntap[4];
    signed char tdy[4][9], tdx[4][9], tid[4][9];
    int ostride, oy[4], ox[4];    // epi_tma: output pixel = tile pixel * ostride + (oy, ox)
    // conv_tc2_kernel, 3x3 stride 1 ("halo" operand): one box per channel chunk holds the tile's pixels WITH their
    // halo, (BH + 2) rows of Wp = W + 2 pixels; tap (kh, kw) reads the 128 rows that start kh * Wp + kw rows further
    // on, so the activations cross L2 -> shared memory once per chunk instead of once per tap.  Accumulator row m is
    // then pixel (m / Wp, m % Wp) of the tile; rows with m % Wp >= W are padding.
    int halo, Wp;
    int a_slots, a_slot_bytes, a_box_bytes;
    unsigned long long *stamp;    // timeline slot of this launch (nullptr: off)
};

struct __align__(8) TcShared {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t aux_full[8];
    uint64_t afull[4], aempty[4];     // halo operand ring of conv_tc2_kernel
    uint32_t tmem_base;
    uint32_t failed;
    RowMap rows;
};

// ---- epilogue through TMA.  One column group (GW accumulator columns) at a time:
//   pass A  thread = accumulator row: tensor memory (+ partner row in shared memory) -> output group in shared memory
//   store   one TMA store of the group
//   pass B  thread = (channel quad, every rpp-th pixel): per-channel sums over the valid pixels of the group
// KA: 0 plain float, 1 plain onto the fixed-point grid, 2 / 3 float coupling + / -, 4 / 5 fixed-point coupling + / -.
// These two passes run once per column group between barriers, on two warps per scheduler: straight-line code that
// is executed once per visit is paid for in instruction fetches, not in issue slots.  So they are kept SMALL (rolled
// loops, the plain conversion instructions) rather than unrolled.
template <int KA>
__device__ __forceinline__ void tma_pass_a(uint32_t tm, int GW, int row, bool valid, const uint8_t *aux, uint8_t *outb, float out_s) {
    const int row_b = GW * 4;
    const int swz = GW == 32 ? (row & 7) : ((row >> 1) & 3);
#pragma unroll 1
    for (int c = 0; c < GW; c += 8) {
        float v[8];
        tmem_ld8(tm + (uint32_t)c, v);
        if (!valid) continue;
#pragma unroll
        for (int j = 0; j < 2; j++) {
            const int off = row * row_b + ((((c >> 2) + j) ^ swz) << 4);
            float4 r = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            if (KA == 2 || KA == 3) {
                const float4 pr = *reinterpret_cast<const float4 *>(aux + off);
                if (KA == 2) { r.x = pr.x + r.x; r.y = pr.y + r.y; r.z = pr.z + r.z; r.w = pr.w + r.w; }
                else { r.x = pr.x - r.x; r.y = pr.y - r.y; r.z = pr.z - r.z; r.w = pr.w - r.w; }
            } else if (KA != 0) {
                int4 iv = make_int4(__float2int_rn(r.x * out_s), __float2int_rn(r.y * out_s), __float2int_rn(r.z * out_s), __float2int_rn(r.w * out_s));
                if (KA >= 4) {
                    const int4 pi = *reinterpret_cast<const int4 *>(aux + off);
                    if (KA == 4) { iv.x = pi.x + iv.x; iv.y = pi.y + iv.y; iv.z = pi.z + iv.z; iv.w = pi.w + iv.w; }
                    else { iv.x = pi.x - iv.x; iv.y = pi.y - iv.y; iv.z = pi.z - iv.z; iv.w = pi.w - iv.w; }
                }
                r = make_float4(__int_as_float(iv.x), __int_as_float(iv.y), __int_as_float(iv.z), __int_as_float(iv.w));
            }
            *reinterpret_cast<float4 *>(outb + off) = r;
        }
    }
}
// KB 0 / 1: sums and second sums of the stored values (float / fixed point); 2 / 3: the two sums of the
// BN+ReLU backward with a float / fixed-point BN input group.  Rows are added in a fixed order.
template <int KB>
__device__ __forceinline__ void tma_pass_b(int GW, const uint8_t *ob, const uint8_t *aux, int jq, int r0, int rpp, int valid_px,
                                           float q, float4 sc4, float4 sh4, float4 mu4, float4 rs4, float (&acc)[8]) {
    const int row_b = GW * 4;
#pragma unroll 1
    for (int pl = r0; pl < valid_px; pl += rpp) {
        const int off = pl * row_b + ((jq ^ (GW == 32 ? (pl & 7) : ((pl >> 1) & 3))) << 4);
        float4 v = *reinterpret_cast<const float4 *>(ob + off);
        if (KB >= 2) {
            float4 tt = *reinterpret_cast<const float4 *>(aux + off);
            if (KB == 3) tt = make_float4(__int2float_rn(__float_as_int(tt.x)) * q, __int2float_rn(__float_as_int(tt.y)) * q,
                                          __int2float_rn(__float_as_int(tt.z)) * q, __int2float_rn(__float_as_int(tt.w)) * q);
            const float dx = fmaf(sc4.x, tt.x, sh4.x) > 0.f ? v.x : 0.f, dy = fmaf(sc4.y, tt.y, sh4.y) > 0.f ? v.y : 0.f;
            const float dz = fmaf(sc4.z, tt.z, sh4.z) > 0.f ? v.z : 0.f, dw = fmaf(sc4.w, tt.w, sh4.w) > 0.f ? v.w : 0.f;
            acc[0] += dx; acc[1] += dy; acc[2] += dz; acc[3] += dw;
            acc[4] += dx * ((tt.x - mu4.x) * rs4.x); acc[5] += dy * ((tt.y - mu4.y) * rs4.y);
            acc[6] += dz * ((tt.z - mu4.z) * rs4.z); acc[7] += dw * ((tt.w - mu4.w) * rs4.w);
        } else {
            if (KB == 1) v = make_float4(__int2float_rn(__float_as_int(v.x)) * q, __int2float_rn(__float_as_int(v.y)) * q,
                                         __int2float_rn(__float_as_int(v.z)) * q, __int2float_rn(__float_as_int(v.w)) * q);
            acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
            acc[4] += v.x * v.x; acc[5] += v.y * v.y; acc[6] += v.z * v.z; acc[7] += v.w * v.w;
        }
    }
}

// Persistent CTA: walks the pixel tiles blockIdx.x, blockIdx.x + gridDim.x, ... of N tile blockIdx.y.
// The operand ring runs on across tiles; the accumulator alternates between two tensor-memory
// buffers so that the epilogue of one tile overlaps the MMAs of the next.
__global__ void __launch_bounds__(kThreadsTma, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_o0, const __grid_constant__ CUtensorMap map_o1,
               const __grid_constant__ CUtensorMap map_x0, const __grid_constant__ CUtensorMap map_x1, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // operand stages first (1024-byte aligned for the 128-byte swizzle), epilogue stage and bookkeeping behind them
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int box_px = p.g.BIMG * p.g.BH * p.g.W;
    const int a_bytes = box_px * p.KC * 2, b_bytes = p.BN * p.KC * 2;
    const int b_off = (128 * p.KC * 2 + 1023) & ~1023;
    const int stage_bytes = b_off + ((b_bytes + 1023) & ~1023);
    // behind the operand ring: the staged epilogue's row stage and running sums, or (epi_tma) the partner ring,
    // two output groups and the running sums per column group
    float *estage = (float *)(tiles + p.stages * stage_bytes);
    const int ng = p.epi_tma ? p.BN / p.GW : 0;
    uint8_t *auxr = (uint8_t *)estage;
    uint8_t *outr = auxr + (p.need_aux ? ng : 0) * p.group_bytes;
    float *gsums = (float *)(outr + 2 * p.group_bytes);
    TcShared *sh = p.epi_tma ? (TcShared *)(gsums + ng * 128 * 8) : (TcShared *)((uint8_t *)estage + kEpiStageBytes + kEpiSumFloats * 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_vt = p.n_cls * p.g.n_px_tiles;     // tiles of all classes
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * p.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; s++) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&sh->acc_full[b], 1); mbar_init(&sh->acc_empty[b], p.epi_tma ? 256 : 128); }
        for (int b = 0; b < 8; b++) mbar_init(&sh->aux_full[b], 1);
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_a); tma_prefetch_desc(&map_b);
        if (p.epi_tma) { tma_prefetch_desc(&map_o0); tma_prefetch_desc(&map_o1); tma_prefetch_desc(&map_x0); tma_prefetch_desc(&map_x1); }
    }
    if (warp == 1) tmem_alloc(&sh->tmem_base, tmem_cols);
    if (warp >= 2) build_row_map(p.g, &sh->rows, ((warp & 3) << 5) | lane);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_enter();             // the set-up above may overlap the kernel before; its outputs are read from here on
    stamp_begin(p.stamp);
    const uint32_t tmem_d = sh->tmem_base;
    const int col0 = blockIdx.y * p.BN;

    // The two single-thread loops below (TMA producer, MMA issuer) set the pace of the whole CTA: a lone thread gets no
    // latency hiding, every instruction costs its full pipeline latency, and a stage's four MMAs take only 256-512
    // clocks.  So no divisions, no table look-ups and no descriptor construction inside them: the ring position is
    // stepped, tap data is read once per tap, descriptors are a base plus increments of the address field.
    if (warp == 0) {
        if (lane == 0) {
            int s = 0; uint32_t round = 0;
            bool ok = true;
            const uint32_t tx = (uint32_t)(a_bytes + b_bytes);
            for (int t = blockIdx.x; t < n_vt && ok; t += gridDim.x) {
                int n0, h0;
                const int cls = t / p.g.n_px_tiles;
                tile_origin(p.g, t - cls * p.g.n_px_tiles, n0, h0);
                const int ntap = p.ntap[cls], hs = h0 * p.stride;
                for (int ti = 0; ti < ntap && ok; ti++) {
                    const int dx = p.tdx[cls][ti], yy = hs + p.tdy[cls][ti];
                    int wc = p.tid[cls][ti] * p.cin_pad;
                    for (int cc = 0; cc < p.cin_pad; cc += p.KC, wc += p.KC) {
                        if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                        uint8_t *sa = tiles + s * stage_bytes;
                        mbar_expect_tx(&sh->full[s], tx);
                        tma_load_4d(sa, &map_a, &sh->full[s], cc, dx, yy, n0);
                        tma_load_2d(sa + b_off, &map_b, &sh->full[s], wc, col0);
                        if (++s == p.stages) { s = 0; round++; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(p.BN);
            const int row_bytes = p.KC * 2, nk = p.KC >> 4;
            const uint64_t da0 = smem_desc(smem_u32(tiles), row_bytes), db0 = smem_desc(smem_u32(tiles) + b_off, row_bytes);
            const uint32_t stage16 = (uint32_t)stage_bytes >> 4;      // the descriptors' address field counts 16-byte units
            int s = 0; uint32_t round = 0, soff = 0;
            bool ok = true;
            int ti = 0;
            for (int t = blockIdx.x; t < n_vt && ok; t += gridDim.x, ti++) {
                const int buf = ti & 1; const uint32_t use = ti >> 1;
                const int iters = p.ntap[t / p.g.n_px_tiles] * p.chunks;
                if (use > 0 && !mbar_wait(&sh->acc_empty[buf], (use - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                tc_fence_after();
                const uint32_t acc = tmem_d + (uint32_t)(buf * p.BN);
                uint32_t accum = 0;
                for (int it = 0; it < iters; it++) {
                    if (!mbar_wait(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = da0 + soff, db = db0 + soff;
                    mma_bf16(acc, da, db, idesc, accum);
                    accum = 1;
                    for (int kk = 1; kk < nk; kk++) mma_bf16(acc, da + 2 * kk, db + 2 * kk, idesc, 1u);
                    mma_commit(&sh->empty[s]);          // frees the stage once these MMAs have read it
                    soff += stage16;
                    if (++s == p.stages) { s = 0; soff = 0; round++; }
                }
                if (ok) mma_commit(&sh->acc_full[buf]);
            }
        }
    } else if (!p.epi_tma) {
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
    } else {
        // epilogue through TMA: two groups of four warps; group wg takes the column groups wg, wg + 2, ... of every
        // tile and owns output slot wg, so that one group's pass over shared memory overlaps the other's waits.
        // Thread etid of a warp group owns accumulator row etid = pixel etid of the tile's box.
        const int wg = (warp - 2) >> 2;
        const int bar_a = 1 + 2 * wg, bar_b = 2 + 2 * wg;   // named barriers of this warp group; 5: both groups
        const int etid = ((warp & 3) << 5) | lane;
        const EpiArgs &e = p.epi;
        const int GW = p.GW, QW = GW >> 2, rpp = 128 / QW;
        const int jq = etid % QW, r0 = etid / QW;
        const int box_px_o = p.g.BIMG * p.g.BH * p.g.W;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const float out_q = e.out.q, out_s = out_q != 0.f ? 1.f / out_q : 0.f, t_q = e.t.q;
        const uint32_t aux_tx = (uint32_t)(box_px_o * GW * 4);
        for (int i = wg * 128 + etid; i < ng * 128 * 8; i += 256) gsums[i] = 0.f;
        // column group gi of this N tile: which tensor of a channel-split pair, and the channel inside it
        auto out_map = [&](int col) { return (p.split_o && col >= p.split_o) ? &map_o1 : &map_o0; };
        auto aux_map = [&](int col) { return (p.split_x && col >= p.split_x) ? &map_x1 : &map_x0; };
        auto col_out = [&](int col) { return (p.split_o && col >= p.split_o) ? col - p.split_o : col; };
        auto col_aux = [&](int col) { return (p.split_x && col >= p.split_x) ? col - p.split_x : col; };
        auto load_aux = [&](int gi, int cls, int n0, int h0) {     // one thread; (cls, n0, h0): class and origin of the tile
            const int col = col0 + gi * GW;
            if (col >= e.n_cols) return;
            mbar_expect_tx(&sh->aux_full[gi], aux_tx);
            tma_load_4d(auxr + gi * p.group_bytes, aux_map(col), &sh->aux_full[gi], col_aux(col), p.ox[cls], h0 * p.ostride + p.oy[cls], n0);
        };
        // class and origin of the tile at hand and of the one after it: worked out once per tile, so that the thread
        // that issues the partner loads between two column groups has no divisions to do
        int cls = 0, n0 = 0, h0 = 0, cls_n = 0, n0_n = 0, h0_n = 0;
        if ((int)blockIdx.x < n_vt) {
            cls_n = (int)blockIdx.x / p.g.n_px_tiles;
            tile_origin(p.g, (int)blockIdx.x - cls_n * p.g.n_px_tiles, n0_n, h0_n);
        }
        if (etid == 0 && p.need_aux && (int)blockIdx.x < n_vt)
            for (int gi = wg; gi < ng; gi += 2) load_aux(gi, cls_n, n0_n, h0_n);
        named_barrier(5, 256);
        bool ok = true;
        int ti = 0;
        uint8_t *ob = outr + wg * p.group_bytes;
        for (int t = blockIdx.x; t < n_vt; t += gridDim.x, ti++) {
            const int buf = ti & 1; const uint32_t use = ti >> 1;
            cls = cls_n; n0 = n0_n; h0 = h0_n;
            const int tn = t + (int)gridDim.x;
            if (tn < n_vt) {
                cls_n = tn / p.g.n_px_tiles;
                tile_origin(p.g, tn - cls_n * p.g.n_px_tiles, n0_n, h0_n);
            }
            const int valid_px = p.g.BIMG > 1 ? (p.g.N - n0 < p.g.BIMG ? p.g.N - n0 : p.g.BIMG) * p.g.BH * p.g.W
                                              : (p.g.H - h0 < p.g.BH ? p.g.H - h0 : p.g.BH) * p.g.W;
            if (etid == 0) ok = mbar_wait(&sh->acc_full[buf], use & 1) && sh->failed == 0;     // one thread polls, the rest block
            ok = named_barrier_and(bar_b, 128, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t tm = tmem_d + lane_base + (uint32_t)(buf * p.BN);
#pragma unroll 1
            for (int gi = wg; gi < ng; gi += 2) {
                const int col = col0 + gi * GW;
                const bool live = col < e.n_cols;          // groups beyond the valid channels only drain their columns
                const uint8_t *ax = auxr + gi * p.group_bytes;
                if (etid == 0) {
                    if (p.need_aux && live) ok = mbar_wait(&sh->aux_full[gi], ti & 1);
                    tma_store_wait_read();                 // this group's last store is done with the output slot
                }
                ok = named_barrier_and(bar_b, 128, ok);
                if (!ok) break;
                const bool rowv = live && etid < valid_px;
                const uint32_t tg = tm + (uint32_t)(gi * GW);
                if (e.mode != EPI_COUPLE) {
                    if (out_q == 0.f) tma_pass_a<0>(tg, GW, etid, rowv, ax, ob, out_s); else tma_pass_a<1>(tg, GW, etid, rowv, ax, ob, out_s);
                } else if (out_q == 0.f) {
                    if (e.sign > 0) tma_pass_a<2>(tg, GW, etid, rowv, ax, ob, out_s); else tma_pass_a<3>(tg, GW, etid, rowv, ax, ob, out_s);
                } else {
                    if (e.sign > 0) tma_pass_a<4>(tg, GW, etid, rowv, ax, ob, out_s); else tma_pass_a<5>(tg, GW, etid, rowv, ax, ob, out_s);
                }
                fence_proxy_async();
                named_barrier(bar_a, 128);
                if (etid == 0 && live) {
                    tma_store_4d(out_map(col), ob, col_out(col), p.ox[cls], h0 * p.ostride + p.oy[cls], n0);
                    tma_store_commit();
                }
                if (e.part && live && col + jq * 4 < e.n_cols) {
                    float4 sc4 = make_float4(0, 0, 0, 0), sh4 = sc4, mu4 = sc4, rs4 = sc4;
                    if (e.mode == EPI_BNBWD) bn_coef4(e.bn, col + jq * 4, sc4, sh4, mu4, rs4);
                    float4 *slot = reinterpret_cast<float4 *>(gsums + (gi * 128 + etid) * 8);
                    const float4 a0 = slot[0], a1 = slot[1];
                    float acc[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                    if (e.mode == EPI_BNBWD) {
                        if (t_q == 0.f) tma_pass_b<2>(GW, ob, ax, jq, r0, rpp, valid_px, 0.f, sc4, sh4, mu4, rs4, acc);
                        else tma_pass_b<3>(GW, ob, ax, jq, r0, rpp, valid_px, t_q, sc4, sh4, mu4, rs4, acc);
                    } else if (out_q == 0.f) tma_pass_b<0>(GW, ob, ax, jq, r0, rpp, valid_px, 0.f, sc4, sh4, mu4, rs4, acc);
                    else tma_pass_b<1>(GW, ob, ax, jq, r0, rpp, valid_px, out_q, sc4, sh4, mu4, rs4, acc);
                    slot[0] = make_float4(acc[0], acc[1], acc[2], acc[3]); slot[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
                }
                named_barrier(bar_a, 128);                 // the partner group and the output slot have been read
                if (etid == 0 && p.need_aux && tn < n_vt) load_aux(gi, cls_n, n0_n, h0_n);
            }
            if (!ok) break;
            // this warp group has drained its columns of the accumulator (the other group arrives for its own)
            tc_fence_before();
            mbar_arrive(&sh->acc_empty[buf]);
        }
        if (etid == 0) tma_store_wait_all();
        if (!ok && lane == 0) atomicExch(&sh->failed, 1u);
        __threadfence_block();
        named_barrier(5, 256);
        if (wg == 0 && e.part && sh->failed == 0) {
            // per-CTA record: the threads that share a channel quad are added in order
            float *mine = e.part + (size_t)blockIdx.x * 2 * e.n_cols;
            for (int gi = 0; gi < ng; gi++) {
                const int col = col0 + gi * GW + jq * 4;
                if (r0 == 0 && col < e.n_cols) {
                    const float *base = gsums + (size_t)gi * 128 * 8;
                    float r[8];
#pragma unroll
                    for (int j = 0; j < 8; j++) r[j] = base[jq * 8 + j];
                    for (int y = 1; y < rpp; y++)
#pragma unroll
                        for (int j = 0; j < 8; j++) r[j] += base[(y * QW + jq) * 8 + j];
                    *reinterpret_cast<float4 *>(mine + 2 * col) = make_float4(r[0], r[1], r[2], r[3]);
                    *reinterpret_cast<float4 *>(mine + 2 * col + 4) = make_float4(r[4], r[5], r[6], r[7]);
                }
            }
            epilogue_publish<128>(e, reinterpret_cast<float *>(auxr), etid);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && sh->failed) atomicExch(p.status, (int)REVNET_E_TIMEOUT);
    stamp_end(p.stamp);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, tmem_cols);
    }
}

// The same convolution on a CTA PAIR (a cluster of two CTAs on the two SMs of a TPC, tcgen05 cta_group::2): one
// MMA of M = 256 covers two adjacent pixel tiles, CTA `rank` holding the operand rows of its own 128 pixels and its
// half of the N tile's weight rows, and receiving its 128 accumulator rows in its own tensor memory.  Per MMA an SM
// then reads 128 x 16 activations and only N/2 x 16 weights from shared memory (and fetches only half of the weight
// tile from L2), which is what lets 256-wide tiles run at the tensor cores' rate instead of the shared-memory port's.
// The leader (rank 0) issues the MMAs for both; each CTA loads its own operands (plain tile loads, no multicast)
// and signals the leader's barrier; commits arrive on the barriers of both CTAs.  Each CTA runs the epilogue of its
// own tile exactly as the single-CTA kernel does (epilogue through TMA only).
// Tile pairs: class c, pair j holds the pixel tiles 2j and 2j + 1 of the class; with an odd tile count the last pair's
// second tile lies outside the tensor (TMA delivers zeros, nothing is stored).
__global__ void __launch_bounds__(kThreadsTma, 1)
conv_tc2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_o0, const __grid_constant__ CUtensorMap map_o1,
                const __grid_constant__ CUtensorMap map_x0, const __grid_constant__ CUtensorMap map_x1, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int box_px = p.g.BIMG * p.g.BH * p.g.W;
    const int BNH = p.BN >> 1;                                   // weight rows this CTA holds
    const int a_bytes = box_px * p.KC * 2, b_bytes = BNH * p.KC * 2;
    const int b_off = (128 * p.KC * 2 + 1023) & ~1023;
    const int stage_bytes = b_off + ((b_bytes + 1023) & ~1023);
    const int ng = p.BN / p.GW;
    // halo mode: the ring holds weight tiles only, the activation boxes have a ring of their own in front of it
    uint8_t *abuf = tiles;
    const int wstage_bytes = (b_bytes + 1023) & ~1023;
    uint8_t *wring = tiles + (p.halo ? p.a_slots * p.a_slot_bytes : 0);
    uint8_t *auxr = p.halo ? wring + p.stages * wstage_bytes : tiles + p.stages * stage_bytes;
    uint8_t *outr = auxr + (p.need_aux ? p.aux_slots : 0) * p.group_bytes;
    float *gsums = (float *)(outr + 2 * p.group_bytes);
    TcShared *sh = (TcShared *)(gsums + ng * 128 * 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = (int)blockIdx.x >> 1, n_pairs = (int)gridDim.x >> 1;
    const int n_pp = (p.g.n_px_tiles + 1) >> 1;                  // tile pairs per class
    const int n_vp = p.n_cls * n_pp;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * p.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; s++) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        // acc_empty (used in the leader): one arrival per epilogue warp group of either CTA
        for (int b = 0; b < 2; b++) { mbar_init(&sh->acc_full[b], 1); mbar_init(&sh->acc_empty[b], 4); }
        for (int b = 0; b < 8; b++) mbar_init(&sh->aux_full[b], 1);
        for (int b = 0; b < 4; b++) { mbar_init(&sh->afull[b], 1); mbar_init(&sh->aempty[b], 1); }
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_a); tma_prefetch_desc(&map_b);
        tma_prefetch_desc(&map_o0); tma_prefetch_desc(&map_o1); tma_prefetch_desc(&map_x0); tma_prefetch_desc(&map_x1);
    }
    if (warp == 1) tmem2_alloc(&sh->tmem_base, tmem_cols);       // the same warp of both CTAs
    if (warp >= 2) build_row_map(p.g, &sh->rows, ((warp & 3) << 5) | lane);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();      // the peer's barriers are initialised and its tensor memory allocated before anything crosses over
    tc_fence_after();
    pdl_enter();
    stamp_begin(p.stamp);
    const uint32_t tmem_d = sh->tmem_base;
    const int col0 = blockIdx.y * p.BN;
    // this CTA's tile of tile pair vp
    auto my_tile = [&](int vp, int &cls, int &t) { cls = vp / n_pp; t = 2 * (vp - cls * n_pp) + (int)rank; };

    // (single-thread loops kept lean, as in conv_tc_kernel)
    if (warp == 0) {
        if (lane == 0) {
            int s = 0, as = 0; uint32_t round = 0, ar = 0;
            bool ok = true;
            const uint32_t full0 = mapa_shared(smem_u32(&sh->full[0]), 0), afull0 = mapa_shared(smem_u32(&sh->afull[0]), 0);   // the leader's barriers
            const uint32_t tx = (uint32_t)(2 * (a_bytes + b_bytes)), txw = (uint32_t)(2 * b_bytes), txa = (uint32_t)(2 * p.a_box_bytes);
            const int wcol = col0 + (int)rank * BNH;
            for (int vp = pair; vp < n_vp && ok; vp += n_pairs) {
                int cls, t, n0, h0;
                my_tile(vp, cls, t);
                tile_origin(p.g, t, n0, h0);         // beyond the last tile the origin lies outside the tensor: zeros arrive
                if (p.halo) {
                    // per channel chunk: one activation box with its halo, then the nine weight tiles
                    for (int cc = 0; cc < p.cin_pad && ok; cc += p.KC) {
                        if (ar > 0 && !mbar_wait(&sh->aempty[as], (ar - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                        if (rank == 0) mbar_expect_tx(&sh->afull[as], txa);
                        tma2_load_4d(abuf + as * p.a_slot_bytes, &map_a, afull0 + 8u * as, cc, -1, h0 - 1, n0);
                        if (++as == p.a_slots) { as = 0; ar++; }
                        int wc = cc;
                        for (int ti = 0; ti < 9; ti++, wc += p.cin_pad) {      // tap ti of a plain 3x3 layer sits at ti * cin_pad in the pack
                            if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                            if (rank == 0) mbar_expect_tx(&sh->full[s], txw);
                            tma2_load_2d(wring + s * wstage_bytes, &map_b, full0 + 8u * s, wc, wcol);
                            if (++s == p.stages) { s = 0; round++; }
                        }
                    }
                    continue;
                }
                const int ntap = p.ntap[cls], hs = h0 * p.stride;
                for (int ti = 0; ti < ntap && ok; ti++) {
                    const int dx = p.tdx[cls][ti], yy = hs + p.tdy[cls][ti];
                    int wc = p.tid[cls][ti] * p.cin_pad;
                    for (int cc = 0; cc < p.cin_pad; cc += p.KC, wc += p.KC) {
                        if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                        uint8_t *sa = tiles + s * stage_bytes;
                        if (rank == 0) mbar_expect_tx(&sh->full[s], tx);      // the leader's barrier collects the bytes of both CTAs
                        tma2_load_4d(sa, &map_a, full0 + 8u * s, cc, dx, yy, n0);
                        tma2_load_2d(sa + b_off, &map_b, full0 + 8u * s, wc, wcol);
                        if (++s == p.stages) { s = 0; round++; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_m256(p.BN);
            const int row_bytes = p.KC * 2, nk = p.KC >> 4;
            const uint64_t da0 = smem_desc(smem_u32(tiles), row_bytes), db0 = smem_desc(smem_u32(tiles) + b_off, row_bytes);
            const uint64_t ha0 = smem_desc(smem_u32(abuf), 128), hb0 = smem_desc(smem_u32(wring), 128);      // halo mode: boxes, weight ring
            const uint32_t stage16 = (uint32_t)stage_bytes >> 4, wstage16 = (uint32_t)wstage_bytes >> 4, aslot16 = (uint32_t)p.a_slot_bytes >> 4;
            const uint32_t wp8 = (uint32_t)p.Wp * 8u;      // one halo row of pixels, in 16-byte units (128-byte operand rows)
            int s = 0, as = 0; uint32_t round = 0, ar = 0, soff = 0, aoff = 0;
            bool ok = true;
            int ti = 0;
            for (int vp = pair; vp < n_vp && ok; vp += n_pairs, ti++) {
                const int buf = ti & 1; const uint32_t use = ti >> 1;
                if (use > 0 && !mbar_wait_cluster(&sh->acc_empty[buf], (use - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                tc_fence_after();
                const uint32_t acc = tmem_d + (uint32_t)(buf * p.BN);
                uint32_t accum = 0;
                if (p.halo) {
                    for (int ch = 0; ch < p.chunks && ok; ch++) {
                        if (!mbar_wait_cluster(&sh->afull[as], ar & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                        // tap (kh, kw): the operand starts kh * Wp + kw rows (of 128 bytes) into the box.  The 128-byte
                        // swizzle is a function of the shared-memory ADDRESS (bits 4..6 xor bits 7..9), for the TMA
                        // write as for the MMA read, so a start on any row reads the rows as they were written
                        uint64_t da_row = ha0 + aoff;
                        for (int kh = 0; kh < 3 && ok; kh++, da_row += wp8) {
                            uint64_t da = da_row;
                            for (int kw = 0; kw < 3; kw++, da += 8) {
                                if (!mbar_wait_cluster(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                                tc_fence_after();
                                const uint64_t db = hb0 + soff;
                                mma2_bf16(acc, da, db, idesc, accum);
                                accum = 1;
                                mma2_bf16(acc, da + 2, db + 2, idesc, 1u);
                                mma2_bf16(acc, da + 4, db + 4, idesc, 1u);
                                mma2_bf16(acc, da + 6, db + 6, idesc, 1u);
                                mma2_commit_both(&sh->empty[s]);
                                soff += wstage16;
                                if (++s == p.stages) { s = 0; soff = 0; round++; }
                            }
                        }
                        if (ok) mma2_commit_both(&sh->aempty[as]);      // the box is free once the MMAs of its nine taps have read it
                        aoff += aslot16;
                        if (++as == p.a_slots) { as = 0; aoff = 0; ar++; }
                    }
                    if (ok) mma2_commit_both(&sh->acc_full[buf]);
                    continue;
                }
                const int iters = p.ntap[vp / n_pp] * p.chunks;
                for (int it = 0; it < iters; it++) {
                    if (!mbar_wait_cluster(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = da0 + soff, db = db0 + soff;
                    mma2_bf16(acc, da, db, idesc, accum);
                    accum = 1;
                    for (int kk = 1; kk < nk; kk++) mma2_bf16(acc, da + 2 * kk, db + 2 * kk, idesc, 1u);
                    mma2_commit_both(&sh->empty[s]);         // frees the stage in both CTAs once these MMAs have read it
                    soff += stage16;
                    if (++s == p.stages) { s = 0; soff = 0; round++; }
                }
                if (ok) mma2_commit_both(&sh->acc_full[buf]);
            }
        }
    } else {
        // epilogue of this CTA's own tile: as in conv_tc_kernel (two groups of four warps, alternate column groups)
        const int wg = (warp - 2) >> 2;
        const int bar_a = 1 + 2 * wg, bar_b = 2 + 2 * wg;
        const int etid = ((warp & 3) << 5) | lane;
        const EpiArgs &e = p.epi;
        const int GW = p.GW, QW = GW >> 2, rpp = 128 / QW;
        const int jq = etid % QW, r0 = etid / QW;
        const int box_px_o = p.g.BIMG * p.g.BH * p.g.W;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const float out_q = e.out.q, out_s = out_q != 0.f ? 1.f / out_q : 0.f, t_q = e.t.q;
        const uint32_t aux_tx = (uint32_t)(box_px_o * GW * 4);
        const uint32_t acc_empty0[2] = {mapa_shared(smem_u32(&sh->acc_empty[0]), 0), mapa_shared(smem_u32(&sh->acc_empty[1]), 0)};
        // pixel of the tile's box (rows of W pixels) this thread's accumulator row holds; -1: padding
        int srow = etid;
        if (p.halo) { const int hh = etid / p.Wp, ww = etid - hh * p.Wp; srow = (hh < p.g.BH && ww < p.g.W) ? hh * p.g.W + ww : -1; }
        const int prow = srow < 0 ? 0 : srow;
        for (int i = wg * 128 + etid; i < ng * 128 * 8; i += 256) gsums[i] = 0.f;
        auto out_map = [&](int col) { return (p.split_o && col >= p.split_o) ? &map_o1 : &map_o0; };
        auto aux_map = [&](int col) { return (p.split_x && col >= p.split_x) ? &map_x1 : &map_x0; };
        auto col_out = [&](int col) { return (p.split_o && col >= p.split_o) ? col - p.split_o : col; };
        auto col_aux = [&](int col) { return (p.split_x && col >= p.split_x) ? col - p.split_x : col; };
        // The partner groups arrive through a ring of SW slots per warp group (slots wg, wg + 2, ...), filled in the
        // order the group will visit them: its column groups of this tile, then of its next tile, ...; groups beyond
        // the valid channels and tiles outside the tensor are not visited.  l_*: next visit to load (one thread),
        // c_*: next visit to consume (all threads, uniform).
        const int SW = p.aux_slots >> 1;
        int l_vp = pair, l_gi = wg, l_slot = 0;
        int c_slot = 0; uint32_t c_par = 0;
        auto load_next_aux = [&]() {                         // one thread; returns without loading once the visits are used up
            while (l_vp < n_vp) {
                int cls, t, n0, h0;
                my_tile(l_vp, cls, t);
                const int col = col0 + l_gi * GW;
                const bool live = col < e.n_cols && t < p.g.n_px_tiles;
                l_gi += 2;
                const bool last_of_tile = l_gi >= ng;
                if (live) {
                    tile_origin(p.g, t, n0, h0);
                    const int slot = wg + 2 * l_slot;
                    mbar_expect_tx(&sh->aux_full[slot], aux_tx);
                    tma_load_4d(auxr + slot * p.group_bytes, aux_map(col), &sh->aux_full[slot], col_aux(col), p.ox[cls], h0 * p.ostride + p.oy[cls], n0);
                    if (++l_slot == SW) l_slot = 0;
                }
                if (last_of_tile) { l_gi = wg; l_vp += n_pairs; }
                if (live) return;
            }
        };
        if (etid == 0 && p.need_aux && wg < ng)
            for (int i = 0; i < SW; i++) load_next_aux();
        named_barrier(5, 256);
        bool ok = true;
        int ti = 0;
        uint8_t *ob = outr + wg * p.group_bytes;
        for (int vp = pair; vp < n_vp; vp += n_pairs, ti++) {
            const int buf = ti & 1; const uint32_t use = ti >> 1;
            int cls, t, n0, h0;
            my_tile(vp, cls, t);
            const bool in_range = t < p.g.n_px_tiles;
            tile_origin(p.g, t, n0, h0);
            int valid_px = 0;
            if (in_range)
                valid_px = p.g.BIMG > 1 ? (p.g.N - n0 < p.g.BIMG ? p.g.N - n0 : p.g.BIMG) * p.g.BH * p.g.W
                                        : (p.g.H - h0 < p.g.BH ? p.g.H - h0 : p.g.BH) * p.g.W;
            if (etid == 0) ok = mbar_wait_cluster(&sh->acc_full[buf], use & 1) && sh->failed == 0;
            ok = named_barrier_and(bar_b, 128, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t tm = tmem_d + lane_base + (uint32_t)(buf * p.BN);
#pragma unroll 1
            for (int gi = wg; gi < ng; gi += 2) {
                const int col = col0 + gi * GW;
                const bool live = in_range && col < e.n_cols;
                const bool visit = p.need_aux && live;       // this group's partner tile sits in ring slot c_slot
                const uint8_t *ax = auxr + (wg + 2 * c_slot) * p.group_bytes;
                if (etid == 0) {
                    if (visit) ok = mbar_wait(&sh->aux_full[wg + 2 * c_slot], c_par);
                    tma_store_wait_read();
                }
                if (visit && ++c_slot == SW) { c_slot = 0; c_par ^= 1u; }
                ok = named_barrier_and(bar_b, 128, ok);
                if (!ok) break;
                const bool rowv = live && srow >= 0 && srow < valid_px;
                const uint32_t tg = tm + (uint32_t)(gi * GW);
                if (e.mode != EPI_COUPLE) {
                    if (out_q == 0.f) tma_pass_a<0>(tg, GW, prow, rowv, ax, ob, out_s); else tma_pass_a<1>(tg, GW, prow, rowv, ax, ob, out_s);
                } else if (out_q == 0.f) {
                    if (e.sign > 0) tma_pass_a<2>(tg, GW, prow, rowv, ax, ob, out_s); else tma_pass_a<3>(tg, GW, prow, rowv, ax, ob, out_s);
                } else {
                    if (e.sign > 0) tma_pass_a<4>(tg, GW, prow, rowv, ax, ob, out_s); else tma_pass_a<5>(tg, GW, prow, rowv, ax, ob, out_s);
                }
                fence_proxy_async();
                named_barrier(bar_a, 128);
                if (etid == 0 && live) {
                    tma_store_4d(out_map(col), ob, col_out(col), p.ox[cls], h0 * p.ostride + p.oy[cls], n0);
                    tma_store_commit();
                }
                if (e.part && live && col + jq * 4 < e.n_cols) {
                    float4 sc4 = make_float4(0, 0, 0, 0), sh4 = sc4, mu4 = sc4, rs4 = sc4;
                    if (e.mode == EPI_BNBWD) bn_coef4(e.bn, col + jq * 4, sc4, sh4, mu4, rs4);
                    float4 *slot = reinterpret_cast<float4 *>(gsums + (gi * 128 + etid) * 8);
                    const float4 a0 = slot[0], a1 = slot[1];
                    float acc[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                    if (e.mode == EPI_BNBWD) {
                        if (t_q == 0.f) tma_pass_b<2>(GW, ob, ax, jq, r0, rpp, valid_px, 0.f, sc4, sh4, mu4, rs4, acc);
                        else tma_pass_b<3>(GW, ob, ax, jq, r0, rpp, valid_px, t_q, sc4, sh4, mu4, rs4, acc);
                    } else if (out_q == 0.f) tma_pass_b<0>(GW, ob, ax, jq, r0, rpp, valid_px, 0.f, sc4, sh4, mu4, rs4, acc);
                    else tma_pass_b<1>(GW, ob, ax, jq, r0, rpp, valid_px, out_q, sc4, sh4, mu4, rs4, acc);
                    slot[0] = make_float4(acc[0], acc[1], acc[2], acc[3]); slot[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
                }
                named_barrier(bar_a, 128);                 // the partner slot and the output slot have been read
                if (etid == 0 && visit) load_next_aux();   // refill the slot just freed
            }
            if (!ok) break;
            // this warp group has drained its columns of the accumulator: one arrival per group on the leader's barrier
            tc_fence_before();
            named_barrier(bar_a, 128);
            if (etid == 0) mbar_arrive_cluster(acc_empty0[buf]);
        }
        if (etid == 0) tma_store_wait_all();
        if (!ok && lane == 0) atomicExch(&sh->failed, 1u);
        __threadfence_block();
        named_barrier(5, 256);
        if (wg == 0 && e.part && sh->failed == 0) {
            float *mine = e.part + (size_t)blockIdx.x * 2 * e.n_cols;
            for (int gi = 0; gi < ng; gi++) {
                const int col = col0 + gi * GW + jq * 4;
                if (r0 == 0 && col < e.n_cols) {
                    const float *base = gsums + (size_t)gi * 128 * 8;
                    float r[8];
#pragma unroll
                    for (int j = 0; j < 8; j++) r[j] = base[jq * 8 + j];
                    for (int y = 1; y < rpp; y++)
#pragma unroll
                        for (int j = 0; j < 8; j++) r[j] += base[(y * QW + jq) * 8 + j];
                    *reinterpret_cast<float4 *>(mine + 2 * col) = make_float4(r[0], r[1], r[2], r[3]);
                    *reinterpret_cast<float4 *>(mine + 2 * col + 4) = make_float4(r[4], r[5], r[6], r[7]);
                }
            }
            epilogue_publish<128>(e, reinterpret_cast<float *>(auxr), etid);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && sh->failed) atomicExch(p.status, (int)REVNET_E_TIMEOUT);
    stamp_end(p.stamp);
    // neither CTA leaves, or frees tensor memory, while the other may still read its operands or signal its barriers
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem2_dealloc(tmem_d, tmem_cols);
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

// all packs of a step in one launch: blockIdx.y walks the job table.  A block (32 x 8 threads) takes tiles of
// 32 rows x 64 columns of the pack (one tap), a thread two adjacent columns: the fp32 reads of a warp are contiguous
// (256 bytes plain, 128 bytes transposed) and so are its bf16x2 writes (128 bytes); the transposed pack goes through
// shared memory.
__global__ void pack_weights_batch_kernel(const PackJob *__restrict__ jobs) {
    pdl_enter();
    __shared__ float tile[64][33];
    const PackJob j = jobs[blockIdx.y];
    const int taps = j.k * j.k;
    const int rt = (j.rows_pad + 31) >> 5, ct = (j.cols_pad + 63) >> 6;
    const int n_tiles = taps * rt * ct;
    const int tx = threadIdx.x, ty = threadIdx.y;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int c0 = (t % ct) << 6, r0 = ((t / ct) % rt) << 5, tap = t / (ct * rt);
        if (!j.transposed) {
#pragma unroll
            for (int rr = 0; rr < 32; rr += 8) {
                const int r = r0 + rr + ty, c = c0 + 2 * tx;      // columns are input channels (a multiple of 4: c and c + 1 are valid together)
                if (r < j.rows_pad && c < j.cols_pad) {
                    float2 v = make_float2(0.f, 0.f);
                    if (r < j.Co && c < j.Ci) v = *reinterpret_cast<const float2 *>(j.W + ((size_t)r * taps + tap) * j.Ci + c);
                    *reinterpret_cast<__nv_bfloat162 *>(j.out + ((size_t)r * taps + tap) * j.cols_pad + c) = __floats2bfloat162_rn(v.x, v.y);
                }
            }
        } else {
            // rows of the pack are input channels, columns output channels, taps mirrored
#pragma unroll
            for (int cc = 0; cc < 64; cc += 8) {
                const int co = c0 + cc + ty, ci = r0 + tx;
                tile[cc + ty][tx] = (co < j.Co && ci < j.Ci) ? j.W[((size_t)co * taps + (taps - 1 - tap)) * j.Ci + ci] : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int rr = 0; rr < 32; rr += 8) {
                const int r = r0 + rr + ty, c = c0 + 2 * tx;
                if (r < j.rows_pad && c < j.cols_pad)
                    *reinterpret_cast<__nv_bfloat162 *>(j.out + ((size_t)r * taps + tap) * j.cols_pad + c) = __floats2bfloat162_rn(tile[2 * tx][rr + ty], tile[2 * tx + 1][rr + ty]);
            }
            __syncthreads();
        }
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
bool tc_shape(Geom g, int cin, int cout, int k, int stride, TcShape &s, bool wide = false) {   // g: output geometry
    if ((stride != 1 && stride != 2) || (k != 1 && k != 3) || cin % 8 || cout % 4) return false;
    if (!tile_geom(g, s.g)) return false;
    if (s.g.W * stride > 256 || s.g.BH * stride > 256) return false;
    s.cin_pad = round_up(cin, 16);
    s.KC = s.cin_pad % 64 == 0 ? 64 : (s.cin_pad % 32 == 0 ? 32 : 16);
    s.chunks = s.cin_pad / s.KC;
    const int cout_pad = round_up(cout, 16);
    s.BN = cout_pad <= 128 ? cout_pad : 128;
    if (wide && cout_pad >= 256) s.BN = 256;        // 128 x 256 tiles: fewer operand bytes per flop
    s.n_tiles = (cout_pad + s.BN - 1) / s.BN;
    const int a_bytes = 128 * s.KC * 2, b_bytes = s.BN * s.KC * 2;
    s.smem = 1024 + 4 * (((a_bytes + 1023) & ~1023) + ((b_bytes + 1023) & ~1023)) + kEpiStageBytes + kEpiSumFloats * 4 + (int)sizeof(TcShared) + 64;
    return true;
}

// act: bf16 [N,H,W,cin]; Wsrc: fp32 weights; transposed selects the dgrad pack
// s2: the data gradient of a 3x3 stride-2 layer.  `act` is then the upstream gradient on the layer's output grid
// (gin), `out` the gradient on the input grid (twice as fine), and the launch's tile list runs over the four parity classes of the
// input pixels: class (py, px) fills the pixels (2i + py, 2j + px) from the taps that reach them,
//   da[2i+py, 2j+px] = sum over th in T(py), tw in T(px) of g[i + th/2, j + tw/2] Wd[th, tw],  T(0) = {1}, T(1) = {0, 2}
// (Wd the mirrored, transposed pack), so the four classes together cost the nine taps once per four pixels.
bool run_conv_tc(Exec &ex, const char *what, const void *act, Geom gin, int cin, int cout, int k, int stride,
                 const float *Wsrc, const bf16 *prepacked, bool transposed, Pair out, Pair partner, int sign, EpiReq req,
                 bool s2 = false) {
    TcShape s;
    if (stride == 2 && (gin.H % 2 || gin.W % 2)) return false;
    if (s2 && (stride != 1 || k != 3 || !transposed || sign || req.stats || out.c1)) return false;
    const Geom g{gin.N, conv_out(gin.H, k, stride), conv_out(gin.W, k, stride)};   // geometry of the tiles
    if (!tc_shape(g, cin, cout, k, stride, s)) return false;
    const int taps = k * k;
    if (!ex.dry && !encoder(ex.ctx)) return false;
    // the taps of every class of this launch
    const int n_cls = s2 ? 4 : 1;
    int ntap[4] = {0, 0, 0, 0}, ntap_all = 0;
    signed char tdy[4][9], tdx[4][9], tid[4][9];
    memset(tdy, 0, sizeof tdy); memset(tdx, 0, sizeof tdx); memset(tid, 0, sizeof tid);
    for (int c = 0; c < n_cls; c++) {
        const int py = c >> 1, px = c & 1;
        for (int th = 0; th < k; th++)
            for (int tw = 0; tw < k; tw++) {
                if (s2 && ((th & 1) == py || (tw & 1) == px)) continue;
                const int i = ntap[c]++;
                tdy[c][i] = (signed char)(s2 ? th / 2 : th - k / 2); tdx[c][i] = (signed char)(s2 ? tw / 2 : tw - k / 2);
                tid[c][i] = (signed char)(th * k + tw);
            }
        ntap_all += ntap[c];
    }
    // epilogue through TMA where a column group never straddles the halves of a channel-split tensor
    const bool need_aux = sign != 0 || req.bnbwd != nullptr;
    const Pair auxp = req.bnbwd ? req.bnbwd->t : partner;
    const int ntap_max = s2 ? 4 : taps;
    // arithmetic-bound layers without a partner tile (transitions, their data gradients): 128 x 256 tiles
    if (!need_aux && !(out.c1 && out.c0 % 32) && (long long)ntap_max * cin >= 1024 && cout >= 256 && cout % 32 == 0) tc_shape(g, cin, cout, k, stride, s, true);
    // 1x1 layers onto 256 channels and more on a CTA pair with 256 x 256 tiles: half the operand traffic from L2 per flop.
    // Measured on the large-image network: layers WITHOUT a partner tile (2048 -> 512 and the like, many channel chunks
    // per tile) 8-12 % faster; layers WITH one (the last layer of a bottleneck function, epilogue-bound, and a partner
    // ring that the wide tile leaves only two slots per warp group) 7-12 % slower.  REVNET_CONV_PAIR1X1 overrides:
    // bit 0 layers with a partner tile, bit 1 layers without (default 2)
    static const bool pair_enabled = [] { const char *v = getenv("REVNET_CONV_PAIR"); return !(v && v[0] == '0'); }();
    static const int pair1x1 = [] { const char *v = getenv("REVNET_CONV_PAIR1X1"); return v ? atoi(v) : 2; }();
    const bool wide1 = k == 1 && stride == 1 && !s2 && cout >= 256 && cout % 32 == 0 && !(out.c1 && out.c0 % 32) &&
                       !(need_aux && auxp.c1 && auxp.c0 % 32) && s.KC == 64 &&
                       pair_enabled && ex.ctx->sm_count % 2 == 0 && s.g.n_px_tiles >= 2 && ((need_aux && (pair1x1 & 1)) || (!need_aux && (pair1x1 & 2)));
    if (wide1) tc_shape(g, cin, cout, k, stride, s, true);
    // 3x3 stride-1 layers with a partner tile (data gradients with the BN-backward sums fused) on a pair: 256-wide tiles
    // too, the partner groups through a ring of two slots per warp group (REVNET_CONV_WIDE3X3=0: 128-wide, as before)
    static const bool wide3_enabled = [] { const char *v = getenv("REVNET_CONV_WIDE3X3"); return !(v && v[0] == '0'); }();
    const bool wide3 = wide3_enabled && k == 3 && stride == 1 && !s2 && need_aux && cout >= 256 && cout % 32 == 0 && !(out.c1 && out.c0 % 32) &&
                       !(auxp.c1 && auxp.c0 % 32) && s.KC == 64 && pair_enabled && ex.ctx->sm_count % 2 == 0 && s.g.n_px_tiles >= 2;
    if (wide3) tc_shape(g, cin, cout, k, stride, s, true);
    // rows of the weight pack (a multiple of its 128-row blocks, whatever the N tile); TMA fills rows beyond with zeros
    const int rp16 = round_up(cout, 16), rows_pad = rp16 <= 128 ? rp16 : round_up(rp16, 128);
    // column groups of 32 floats, or of 16 where the N tile or the halves of a channel-split tensor ask for it
    int GW = s.BN % 32 == 0 ? 32 : 16;
    if (GW == 32 && s.BN <= 128 && ((out.c1 && out.c0 % 32) || (need_aux && auxp.c1 && auxp.c0 % 32))) GW = 16;
    const int ng = s.BN / GW, group_bytes = (128 * GW * 4 + 1023) & ~1023;
    bool epi_tma = !(out.c1 && out.c0 % GW) && !(need_aux && auxp.c1 && auxp.c0 % GW) && ng <= 8;
    const int ostride = s2 ? 2 : 1;
    if (s2 && (!epi_tma || g.W * 2 > 256 || s.g.BH * 2 > 256)) return false;
    int stages = 4;
    // CTA pairs (conv_tc2_kernel) wherever the epilogue runs through TMA, the N tile splits into two halves of whole
    // 16-row groups and there are at least two pixel tiles; REVNET_CONV_PAIR=0 keeps the single-CTA kernel (for comparison)
    // (1x1 layers are bound by the activations' way from HBM, which a pair does not shorten: measured 3-10 % slower there)
    bool pair = pair_enabled && epi_tma && (k == 3 || wide1) && s.BN % 32 == 0 && s.BN >= 64 && s.g.n_px_tiles >= 2 && ex.ctx->sm_count % 2 == 0;
    // partner ring of the pair kernel: per epilogue warp group as many slots as it has column groups in a tile (at most 4)
    int aux_slots = 0;
    if (need_aux) { int sw = (ng + 1) / 2; if (sw > 4) sw = 4; aux_slots = 2 * sw; }
    // 3x3 stride-1 layers on a pair: the activations of a tile arrive once per channel chunk as one box with its halo
    // (see TcParams::halo); needs 64-channel chunks (128-byte operand rows) and tiles of whole image rows
    static const bool halo_enabled = [] { const char *v = getenv("REVNET_CONV_HALO"); return !(v && v[0] == '0'); }();
    bool halo = halo_enabled && pair && k == 3 && stride == 1 && !s2 && s.KC == 64 && s.g.BIMG == 1 && g.W + 2 <= 128;
    int a_slot_bytes = 0, a_box_bytes = 0;
    const int a_slots = 2;
    if (halo) {
        const int Wp = g.W + 2;
        int bh = 128 / Wp; if (bh > g.H) bh = g.H;
        s.g.BH = bh;
        s.g.tiles_per_img = (g.H + bh - 1) / bh;
        s.g.n_px_tiles = g.N * s.g.tiles_per_img;
        const int box_rows = (bh + 2) * Wp, read_rows = 2 * Wp + 2 + 128;       // rows the box holds / rows the last tap reads up to
        a_box_bytes = box_rows * 128;
        a_slot_bytes = ((box_rows > read_rows ? box_rows : read_rows) * 128 + 1023) & ~1023;
    }
    if (epi_tma) {
        stages = kStages;
        auto stage_bytes_of = [&](bool pr) {
            if (halo) return ((s.BN / 2) * s.KC * 2 + 1023) & ~1023;           // weight tiles only; the boxes are counted below
            return ((128 * s.KC * 2 + 1023) & ~1023) + (((pr ? s.BN / 2 : s.BN) * s.KC * 2 + 1023) & ~1023);
        };
        auto smem_of = [&](int st, bool pr) { return 1024 + (halo ? a_slots * a_slot_bytes : 0) + st * stage_bytes_of(pr) + ((need_aux ? (pr ? aux_slots : ng) : 0) + 2) * group_bytes + ng * 128 * 32 + (int)sizeof(TcShared) + 64; };
        // what does not fit gives way in this order: operand stages down to 3, partner slots down to 2 per warp group, stages down to 2
        while (stages > 3 && smem_of(stages, pair) > 227 * 1024) stages--;
        while (pair && aux_slots > 4 && smem_of(stages, pair) > 227 * 1024) aux_slots -= 2;
        while (stages > 2 && smem_of(stages, pair) > 227 * 1024) stages--;
        if (smem_of(stages, pair) > 227 * 1024) {
            if (s.BN == 256) return false;      // (does not happen: three stages of a wide tile fit)
            epi_tma = false; pair = false; stages = 4;
            if (halo) { halo = false; tile_geom(g, s.g); }
        } else s.smem = smem_of(stages, pair);
    }
    if ((s2 || s.BN == 256) && !epi_tma) return false;
    ex.flops += 2ull * g.P() * cout * cin * ntap_all;
    int occ = (227 * 1024) / s.smem; if (occ > 2) occ = 2; if (occ < 1) occ = 1;
    int ctas = ex.ctx->sm_count * occ / s.n_tiles; if (ctas < 1) ctas = 1;
    if (ctas > s.g.n_px_tiles * n_cls) ctas = s.g.n_px_tiles * n_cls;
    if (pair) {
        // one pair per TPC and N tile; a pair walks tile pairs
        const int n_vp = n_cls * ((s.g.n_px_tiles + 1) / 2);
        int pairs = (ex.ctx->sm_count / 2) / s.n_tiles; if (pairs < 1) pairs = 1;
        if (pairs > n_vp) pairs = n_vp;
        ctas = 2 * pairs;
    }
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
            if (halo) { box[1] = (cuuint32_t)(g.W + 2); box[2] = (cuuint32_t)(s.g.BH + 2); }
            cuuint32_t es[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
            CUresult r = enc(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, (void *)act, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) { ex.failed = true; ex.ctx->err = std::string(what) + ": tensor map (activations) rejected"; ex.ws.release(m); return true; }
        }
        {
            cuuint64_t dims[2] = {(cuuint64_t)taps * s.cin_pad, (cuuint64_t)rows_pad};
            cuuint64_t strides[1] = {(cuuint64_t)taps * s.cin_pad * 2};
            cuuint32_t box[2] = {(cuuint32_t)s.KC, (cuuint32_t)(pair ? s.BN / 2 : s.BN)};     // a CTA of a pair loads its half of the N tile
            cuuint32_t es[2] = {1, 1};
            CUresult r = enc(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void *)wp, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) { ex.failed = true; ex.ctx->err = std::string(what) + ": tensor map (weights) rejected"; ex.ws.release(m); return true; }
        }
        CUtensorMap map_o[2], map_x[2];
        memset(map_o, 0, sizeof map_o); memset(map_x, 0, sizeof map_x);
        if (epi_tma) {
            const CUtensorMapSwizzle gsw = GW == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
            auto enc_f32 = [&](CUtensorMap *map, const float *base, int C) {
                // the epilogue's tensors live on the output grid: the tile's grid, or (parity class) the twice finer
                // one walked with stride 2
                const cuuint64_t Wo = (cuuint64_t)g.W * ostride, Ho = (cuuint64_t)g.H * ostride;
                cuuint64_t dims[4] = {(cuuint64_t)C, Wo, Ho, (cuuint64_t)g.N};
                cuuint64_t strides[3] = {(cuuint64_t)C * 4, Wo * C * 4, Ho * Wo * C * 4};
                cuuint32_t box[4] = {(cuuint32_t)GW, (cuuint32_t)(g.W * ostride), (cuuint32_t)(s.g.BH * ostride), (cuuint32_t)s.g.BIMG};
                cuuint32_t es[4] = {1, (cuuint32_t)ostride, (cuuint32_t)ostride, 1};
                return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, (void *)base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           gsw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
            };
            bool ok = enc_f32(&map_o[0], out.p0, out.c0);
            if (out.c1) ok = ok && enc_f32(&map_o[1], out.p1, out.c1); else map_o[1] = map_o[0];
            if (need_aux) {
                ok = ok && enc_f32(&map_x[0], auxp.p0, auxp.c0);
                if (auxp.c1) ok = ok && enc_f32(&map_x[1], auxp.p1, auxp.c1); else map_x[1] = map_x[0];
            } else { map_x[0] = map_x[1] = map_o[0]; }
            if (!ok) { ex.failed = true; ex.ctx->err = std::string(what) + ": tensor map (epilogue) rejected"; ex.ws.release(m); return true; }
        }
        TcParams p;
        p.stages = stages; p.epi_tma = epi_tma ? 1 : 0; p.GW = GW; p.group_bytes = group_bytes; p.need_aux = need_aux ? 1 : 0;
        p.aux_slots = aux_slots;
        p.split_o = out.c1 ? out.c0 : 0; p.split_x = (need_aux && auxp.c1) ? auxp.c0 : 0;
        memcpy(p.ntap, ntap, sizeof ntap); memcpy(p.tdy, tdy, sizeof tdy); memcpy(p.tdx, tdx, sizeof tdx); memcpy(p.tid, tid, sizeof tid);
        p.ostride = ostride; p.n_cls = n_cls;
        p.halo = halo ? 1 : 0; p.Wp = g.W + 2; p.a_slots = a_slots; p.a_slot_bytes = a_slot_bytes; p.a_box_bytes = a_box_bytes;
        for (int c = 0; c < 4; c++) { p.oy[c] = s2 ? c >> 1 : 0; p.ox[c] = s2 ? c & 1 : 0; }
        p.taps = taps; p.k = k; p.chunks = s.chunks; p.KC = s.KC; p.cin_pad = s.cin_pad; p.BN = s.BN; p.stride = stride; p.g = s.g;
        p.status = ex.ctx->dev_status;
        p.stamp = ex.stamp_slot();
        EpiArgs &e = p.epi;
        memset(&e, 0, sizeof e);
        e.mode = req.bnbwd ? EPI_BNBWD : (sign ? EPI_COUPLE : EPI_PLAIN);
        e.out = out; e.partner = partner; e.sign = sign; e.n_cols = cout; e.pitch = kEpiPitch;
        e.part = part; e.counter = reduce ? ex.ctx->counter() : nullptr;
        e.inv_count = 1.0 / ((double)g.P() * ostride * ostride); e.eps = ex.eps;     // pixels of the output grid
        if (req.stats) { e.mean = req.stats->mean; e.rstd = req.stats->rstd; }
        if (req.bnbwd) { e.t = req.bnbwd->t; e.bn = req.bnbwd->bn; e.dgamma = req.bnbwd->dgamma; e.dbeta = req.bnbwd->dbeta; e.coef = req.bnbwd->coef; }
        static OncePerDevice once;
        if (once.first(ex.ctx->device)) {
            cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
            cudaFuncSetAttribute(conv_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        }
        dim3 grid((unsigned)ctas, (unsigned)s.n_tiles);
        if (pair) launch_cluster(ex, conv_tc2_kernel, grid, kThreadsTma, s.smem, 2, map_a, map_b, map_o[0], map_o[1], map_x[0], map_x[1], p);
        else launch(ex, conv_tc_kernel, grid, epi_tma ? kThreadsTma : kThreads, s.smem, map_a, map_b, map_o[0], map_o[1], map_x[0], map_x[1], p);
        const double bytes = (double)gin.P() * cin * 2 + (double)g.P() * cout * (sign || req.bnbwd ? 8 : 4) + (double)cout * taps * cin * 2;
        // (records of launches on a CTA pair carry the pair kernel's name)
        ex.check(!pair ? what : (transposed ? "conv_dgrad_tc2" : "conv_fprop_tc2"), bytes, 2.0 * g.P() * cout * cin * ntap_all);
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
    int pair;                    // wgrad_tc2_kernel: BN is what ONE CTA of a pair holds of the pair's 2 * BN output channels,
                                 // GM the pair's M groups of 256 rows (CTA r takes the 128-row groups 2j + r of the chunk)
};

// One launch computes the weight gradients of up to kWgMaxJobs layers: each CTA finds its job from
// its index and then works on that layer alone.
constexpr int kWgMaxJobs = 4;
struct alignas(64) WgJob { CUtensorMap map_a, map_g; WgParams p; };
struct WgBatch { WgJob job[kWgMaxJobs]; int n; unsigned long long *stamp; };

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
    stamp_begin(batch.stamp);
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
        int s = 0; uint32_t round = 0;
        for (int it = 0; it < my_tiles; it++) {
            bool ok = true;
            if (lane == 0) {
                if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; }
                if (ok) mbar_expect_tx(&sh->full[s], tx);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const int t = split + it * p.splits;
            const int n0 = p.BIMG > 1 ? t * p.BIMG : t / tiles_per_img;
            const int h0 = p.BIMG > 1 ? 0 : (t - n0 * tiles_per_img) * p.BH;
            uint8_t *sa = tiles + s * stage_bytes;
            if (a_lane) tma_load_4d(sa + lane * blk_bytes_a, &map_a, &sh->full[s], cb * p.blockC, kw - pad, h0 * p.stride + kh - pad, n0);
            else if (g_lane) tma_load_4d(sa + a_region + bg * blk_bytes_b, &map_g, &sh->full[s], g_c, g_x, h0, n0);
            if (++s == p.stages) { s = 0; round++; }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(p.BN, true);
            const int rba = p.blockC * 2, rbb = p.blockN * 2;
            // one thread issues everything: descriptors are a base plus increments of the address field (16-byte units),
            // the ring position is stepped (no divisions in the loop)
            const uint64_t da0 = smem_desc_mn(smem_u32(tiles), rba, blk_bytes_a), db0 = smem_desc_mn(smem_u32(tiles) + a_region, rbb, blk_bytes_b);
            const uint32_t stage16 = (uint32_t)stage_bytes >> 4;
            int s = 0; uint32_t round = 0, soff = 0;
            for (int it = 0; it < my_tiles; it++) {
                if (!mbar_wait(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t accum = it > 0 ? 1u : 0u;
                for (int g = 0; g < groups; g++) {
                    uint64_t da = da0 + soff + (uint32_t)(g * 2048), db = db0 + soff;      // an M group is 32 KB from its first block
                    const uint32_t acc = tmem_d + (uint32_t)(g * p.BN);
                    mma_bf16(acc, da, db, idesc, accum);
                    for (int ks = 1; ks < 8; ks++) {         // 16 pixels per MMA
                        da += (uint32_t)rba; db += (uint32_t)rbb;
                        mma_bf16(acc, da, db, idesc, 1u);
                    }
                }
                mma_commit(&sh->empty[s]);
                soff += stage16;
                if (++s == p.stages) { s = 0; soff = 0; round++; }
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
    stamp_end(batch.stamp);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, tmem_cols);
    }
}

// The same on a CTA pair (tcgen05 cta_group::2): an MMA of M = 256 covers two 128-row groups of (tap, input channel) rows,
// CTA `rank` holding the activation blocks of the groups 2j + rank and HALF of the pair's gradient channels; N = 2 * BN.
// Per pixel tile a CTA then loads GM x 32 KB of activations and BN x 256 B of gradients for GM x 8 MMAs of 256 x 2BN:
// half the operand bytes per flop of the single-CTA form, whose 94 bytes per MMA clock are more than an SM can take in.
// Not for the tap-split (sep) form.  Launched as clusters of two; every job of a launch is of this kind.
__global__ void __launch_bounds__(kThreads, 1)
wgrad_tc2_kernel(const __grid_constant__ WgBatch batch) {
    int jb = 0;
    while (jb + 1 < batch.n && (int)blockIdx.x >= batch.job[jb + 1].p.cta0) jb++;
    const WgParams &p = batch.job[jb].p;
    const CUtensorMap &map_a = batch.job[jb].map_a, &map_g = batch.job[jb].map_g;
    const uint32_t rank = cluster_ctarank();
    const int local = ((int)blockIdx.x - p.cta0) >> 1;         // pair index inside the job (cta0 is even)
    const int split = local % p.splits, chunk = (local / p.splits) % p.m_chunks, ntile = local / (p.splits * p.m_chunks);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int blk_bytes_a = 256 * p.blockC, blk_bytes_b = 256 * p.blockN;   // [128 pixels][block] bf16
    const int a_region = p.GM * 32768;                         // whole groups: 32 KB each
    const int stage_bytes = a_region + ((256 * p.BN + 1023) & ~1023);
    TcShared *sh = (TcShared *)(tiles + p.stages * stage_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bpg = 128 / p.blockC;                          // blocks per 128-row group
    const int first_block = chunk * 2 * p.GM * bpg;          // the pair's chunk: 2 * GM groups
    // blocks this CTA / the other CTA loads per pixel tile: group 2j + r holds the blocks first_block + (2j + r) * bpg ...
    auto blocks_of = [&](int r) { int n = 0; for (int j = 0; j < p.GM; j++) { int b = p.total_blocks - (first_block + (2 * j + r) * bpg); n += b < 0 ? 0 : (b > bpg ? bpg : b); } return n; };
    const int col0 = ntile * 2 * p.BN;                       // first output channel of the pair's N tile
    auto nblocks_of = [&](int r) { int n = (p.cout - (col0 + r * p.BN) + p.blockN - 1) / p.blockN; return n < 0 ? 0 : (n > p.BN / p.blockN ? p.BN / p.blockN : n); };
    const int my_tiles = (p.n_tiles_px - split + p.splits - 1) / p.splits;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < p.GM * 2 * p.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; s++) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        mbar_init(&sh->acc_full[0], 1);
        sh->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem2_alloc(&sh->tmem_base, tmem_cols);
    {
        // rows and blocks TMA never writes (short tiles, groups beyond the last block) must hold zeros, not stale bits:
        // their products land in rows that are never stored, but a NaN pattern would still be a NaN
        uint4 *z = reinterpret_cast<uint4 *>(tiles);
        const int n16 = p.stages * stage_bytes / 16;
        for (int i = threadIdx.x; i < n16; i += kThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    pdl_enter();
    stamp_begin(batch.stamp);
    const uint32_t tmem_d = sh->tmem_base;
    const int pad = p.k / 2;
    const int tiles_per_img = p.tiles_per_img;

    if (warp == 0) {
        // lane (j, i) with j < GM, i < bpg: activation block i of this CTA's group 2j + rank; the next lanes: gradient blocks
        const uint32_t tx = (uint32_t)(p.box_px * 2 * ((blocks_of(0) + blocks_of(1)) * p.blockC + (nblocks_of(0) + nblocks_of(1)) * p.blockN));
        const int nb_n = nblocks_of((int)rank);
        const int ja = lane / bpg, ia = lane - ja * bpg;
        const int gb = first_block + (2 * ja + (int)rank) * bpg + ia;
        const bool a_lane = lane < p.GM * bpg && gb < p.total_blocks;
        const int tap = gb / p.cblks, cb = gb - tap * p.cblks;
        const int kh = tap / p.k, kw = tap - kh * p.k;
        const int bg = lane - p.GM * bpg;
        const bool g_lane = bg >= 0 && bg < nb_n;
        const int g_c = col0 + (int)rank * p.BN + bg * p.blockN;
        const uint32_t full0 = mapa_shared(smem_u32(&sh->full[0]), 0);
        int s = 0; uint32_t round = 0;
        for (int it = 0; it < my_tiles; it++) {
            bool ok = true;
            if (lane == 0) {
                if (round > 0 && !mbar_wait(&sh->empty[s], (round - 1) & 1)) { atomicExch(&sh->failed, 1u); ok = false; }
                if (ok && rank == 0) mbar_expect_tx(&sh->full[s], tx);       // the leader's barrier collects the bytes of both CTAs
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const int t = split + it * p.splits;
            const int n0 = p.BIMG > 1 ? t * p.BIMG : t / tiles_per_img;
            const int h0 = p.BIMG > 1 ? 0 : (t - n0 * tiles_per_img) * p.BH;
            uint8_t *sa = tiles + s * stage_bytes;
            if (a_lane) tma2_load_4d(sa + ja * 32768 + ia * blk_bytes_a, &map_a, full0 + 8u * s, cb * p.blockC, kw - pad, h0 * p.stride + kh - pad, n0);
            else if (g_lane) tma2_load_4d(sa + a_region + bg * blk_bytes_b, &map_g, full0 + 8u * s, g_c, 0, h0, n0);
            if (++s == p.stages) { s = 0; round++; }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_m256(2 * p.BN) | (3u << 15);     // both operands M / N-major
            const int rba = p.blockC * 2, rbb = p.blockN * 2;
            const uint64_t da0 = smem_desc_mn(smem_u32(tiles), rba, blk_bytes_a), db0 = smem_desc_mn(smem_u32(tiles) + a_region, rbb, blk_bytes_b);
            const uint32_t stage16 = (uint32_t)stage_bytes >> 4;
            int s = 0; uint32_t round = 0, soff = 0;
            for (int it = 0; it < my_tiles; it++) {
                if (!mbar_wait_cluster(&sh->full[s], round & 1)) { atomicExch(&sh->failed, 1u); break; }
                tc_fence_after();
                const uint32_t accum = it > 0 ? 1u : 0u;
                for (int g = 0; g < p.GM; g++) {
                    uint64_t da = da0 + soff + (uint32_t)(g * 2048), db = db0 + soff;
                    const uint32_t acc = tmem_d + (uint32_t)(g * 2 * p.BN);
                    mma2_bf16(acc, da, db, idesc, accum);
                    for (int ks = 1; ks < 8; ks++) {         // 16 pixels per MMA
                        da += (uint32_t)rba; db += (uint32_t)rbb;
                        mma2_bf16(acc, da, db, idesc, 1u);
                    }
                }
                mma2_commit_both(&sh->empty[s]);
                soff += stage16;
                if (++s == p.stages) { s = 0; soff = 0; round++; }
            }
            mma2_commit_both(&sh->acc_full[0]);
        }
    } else {
        const int quarter = warp & 3;
        bool ok = true;
        if (quarter == 0 && lane == 0) ok = mbar_wait_cluster(&sh->acc_full[0], 0);
        ok = named_barrier_and(2, 128, ok);
        tc_fence_after();
        if (ok && sh->failed == 0) {
            const int m = quarter * 32 + lane;
            float *dst = p.partial + (size_t)split * p.slice;
            for (int g = 0; g < p.GM; g++) {
                const int gb = first_block + (2 * g + (int)rank) * bpg + m / p.blockC;
                const int tap = gb / p.cblks, ci = (gb - tap * p.cblks) * p.blockC + m % p.blockC;
                const bool row_ok = gb < p.total_blocks && ci < p.cin;
                for (int c = 0; c < 2 * p.BN; c += 16) {
                    float v[16];
                    tmem_ld16(tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(g * 2 * p.BN + c), v);   // whole warp takes part
                    if (!row_ok) continue;
                    if (my_tiles == 0) {
#pragma unroll
                        for (int j = 0; j < 16; j++) v[j] = 0.f;
                    }
                    const int cb0 = col0 + c;
                    if (p.splits > 1) {
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
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && sh->failed) atomicExch(p.status, (int)REVNET_E_TIMEOUT);
    stamp_end(batch.stamp);
    cluster_sync_all();      // neither CTA leaves, or frees tensor memory, while the other may still read its operands
    if (warp == 1) {
        tc_fence_after();
        tmem2_dealloc(tmem_d, tmem_cols);
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

// The same sum for large gradients: 32 x 32 tiles ((tap, ci) rows x output channels) through shared memory, so that
// the reads of the partials (output channels contiguous) and the writes of dW ((tap, ci) contiguous) are both whole
// lines; a thread adds the splits of its four elements in ascending order, four loads in flight per element.
__global__ void __launch_bounds__(256) splitk_sum_tiled_kernel(const SumBatch b) {
    pdl_enter();
    __shared__ float tile[32][33];
    const int j = blockIdx.y;
    const float *__restrict__ part = b.part[j];
    const size_t n = b.n[j];
    const int splits = b.splits[j], C = b.cout[j], R = b.rows[j];
    const int tc_n = (C + 31) >> 5, tr_n = (R + 31) >> 5;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int t = blockIdx.x; t < tc_n * tr_n; t += gridDim.x) {
        const int c0 = (t % tc_n) << 5, r0 = (t / tc_n) << 5;
#pragma unroll
        for (int k = 0; k < 4; k++) {
            const int row = r0 + ty + 8 * k, co = c0 + tx;
            float s = 0.f;
            if (row < R && co < C) {
                const float *src = part + (size_t)row * C + co;
                int z = 0;
                for (; z + 4 <= splits; z += 4) {
                    const float v0 = src[(size_t)z * n], v1 = src[(size_t)(z + 1) * n], v2 = src[(size_t)(z + 2) * n], v3 = src[(size_t)(z + 3) * n];
                    s += v0; s += v1; s += v2; s += v3;
                }
                for (; z < splits; z++) s += src[(size_t)z * n];
            }
            tile[ty + 8 * k][tx] = s;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 4; k++) {
            const int co = c0 + ty + 8 * k, row = r0 + tx;
            if (row < R && co < C) b.out[j][(size_t)co * R + row] = tile[tx][ty + 8 * k];
        }
        __syncthreads();
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


// Data gradient of a 3x3 stride-2 layer: one launch whose tile list runs over the four parity classes of the input
// pixels (see run_conv_tc).  g: bf16 [N, H/2, W/2, cout]; da: fp32 [N, H, W, cin]; bb: BN-backward sums to fuse.
// Large layers (those that get 128 x 256 tiles when no partner tile has to fit beside the operand ring) leave the
// sums to their own pass instead: *fused tells which.
bool conv_dgrad_tc_s2(Exec &ex, const void *g, Geom gi, const Layer &L, float *da, const BnBwdReq *bb, bool *fused) {
    if (L.stride != 2 || L.k != 3 || gi.H % 2 || gi.W % 2) return false;
    const Geom go{gi.N, gi.H / 2, gi.W / 2};
    const bool wide = 4ll * L.cout >= 1024 && L.cin >= 256 && L.cin % 32 == 0;
    EpiReq req; req.bnbwd = wide ? nullptr : bb;
    *fused = req.bnbwd != nullptr;
    return run_conv_tc(ex, "conv_dgrad_tc", g, go, L.cout, L.cin, 3, 1, L.W, L.Wp_dgrad, true, single(da, L.cin), Pair{}, 0, req, true);
}

constexpr int kWgSmemMax = 224 * 1024;

// Shape decisions of one layer's weight gradient; cta_budget: the CTAs the job may take
struct WgPlan { WgParams p; Geom go; int n_tiles, stage_bytes, tail_bytes; };
// pair: plan for wgrad_tc2_kernel (cta_budget then counts CTAs too; the job takes an even number)
static bool wgrad_plan(Geom gi, const Layer &L, int cta_budget, WgPlan &w, bool allow_sep = true, bool pair = false) {
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
    p.sep = (allow_sep && !pair && L.k == 3 && L.stride == 1 && 3 * cin_pad <= 128 && 3 * cout_pad <= 256 && 2 * bpg + 3 * (cout_pad / p.blockN) <= 32) ? 1 : 0;
    p.pair = pair ? 1 : 0;
    if (pair) {
        // a pair's N tile is 2 * BN wide (BN per CTA, a whole number of gradient blocks), its M chunk 2 * GM groups
        // (N tiles of less than 256 columns measured slower on a pair than 128-column tiles on one CTA: 89 against 72 us
        // for the 3x3 layer of 128 channels at 56 x 56, batch 64)
        if (cout_pad < 256 || cout_pad % 32) return false;
        p.total_blocks = taps * p.cblks;
        p.BN = 128;
        if (p.BN % p.blockN) { p.blockN = pick_block(p.BN); if (p.BN % p.blockN) return false; }
        const int groups_all = (p.total_blocks + bpg - 1) / bpg;
        if (groups_all < 2) return false;
        p.GM = groups_all >= 4 ? 2 : 1;
        p.m_chunks = (groups_all + 2 * p.GM - 1) / (2 * p.GM);
        w.n_tiles = (cout_pad + 2 * p.BN - 1) / (2 * p.BN);
        p.H = w.go.H; p.W = w.go.W; p.stride = L.stride;
        p.n_tiles_px = tg.n_px_tiles;
        p.a_region = p.GM * 32768;
        w.stage_bytes = p.a_region + ((256 * p.BN + 1023) & ~1023);
        w.tail_bytes = 0;
        p.stages = (kWgSmemMax - 2048) / w.stage_bytes; if (p.stages > kWgStages) p.stages = kWgStages;
        if (p.stages < 2) return false;
        const int units = p.m_chunks * w.n_tiles, budget = cta_budget / 2 < 1 ? 1 : cta_budget / 2;     // in pairs
        auto clampi = [&](int v) { return v < 1 ? 1 : (v > p.n_tiles_px ? p.n_tiles_px : v); };
        const int s_hi = clampi((budget + units - 1) / units), s_lo = clampi(budget / units);
        auto serial_tiles = [&](int sp) { return ((units * sp + budget - 1) / budget) * ((p.n_tiles_px + sp - 1) / sp); };
        p.splits = serial_tiles(s_lo) < serial_tiles(s_hi) ? s_lo : s_hi;
        p.slice = (size_t)L.cout * taps * L.cin;
        return true;
    }
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
    p.stages = (kWgSmemMax - 2048 - w.tail_bytes) / w.stage_bytes; if (p.stages > kWgStages) p.stages = kWgStages;
    if (p.stages < 2) return p.sep ? wgrad_plan(gi, L, cta_budget, w, false) : false;
    // split the pixel reduction so that the job's CTAs cover its share of the machine once: rounding the split
    // count up may spill a few CTAs into a second wave (these CTAs fill an SM each), rounding down leaves SMs idle;
    // take whichever walks fewer pixel tiles one after the other
    const int pairs = p.m_chunks * w.n_tiles;
    auto clampi = [&](int v) { return v < 1 ? 1 : (v > p.n_tiles_px ? p.n_tiles_px : v); };
    const int s_hi = clampi((cta_budget + pairs - 1) / pairs), s_lo = clampi(cta_budget / pairs);
    auto serial_tiles = [&](int sp) { return ((pairs * sp + cta_budget - 1) / cta_budget) * ((p.n_tiles_px + sp - 1) / sp); };
    int splits = serial_tiles(s_lo) < serial_tiles(s_hi) ? s_lo : s_hi;
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
    // CTA pairs (wgrad_tc2_kernel) when every layer of the launch takes them: a launch is made of clusters or it is not
    static const bool pair_enabled = [] { const char *v = getenv("REVNET_WGRAD_PAIR"); return !(v && v[0] == '0'); }();
    bool pair = pair_enabled && ex.ctx->sm_count % 2 == 0;
    for (int j = 0; j < n && pair; j++) pair = wgrad_plan(gi[j], *L[j], budget & ~1, w[j], false, true);
    for (int j = 0; j < n; j++) {
        if (!pair && !wgrad_plan(gi[j], *L[j], budget, w[j])) return false;
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
        batch.stamp = ex.stamp_slot();
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
            cta += p.splits * p.m_chunks * w[j].n_tiles * (pair ? 2 : 1);
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
        static OncePerDevice once;
        if (once.first(ex.ctx->device)) {
            cudaFuncSetAttribute(wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kWgSmemMax);
            cudaFuncSetAttribute(wgrad_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kWgSmemMax);
        }
        if (pair) launch_cluster(ex, wgrad_tc2_kernel, (unsigned)cta, kThreads, smem, 2, batch);
        else launch(ex, wgrad_tc_kernel, (unsigned)cta, kThreads, smem, batch);
        ex.check(pair ? "conv_wgrad_tc2" : "conv_wgrad_tc", bytes, flops);
        if (n_sums) {
            if (max_slice >= 524288) {
                size_t tiles = (max_slice + 1023) / 1024; if (tiles > (size_t)ex.ctx->sm_count * 8) tiles = (size_t)ex.ctx->sm_count * 8;
                dim3 grid((unsigned)tiles, (unsigned)n_sums);
                launch(ex, splitk_sum_tiled_kernel, grid, 256, 0, sums);
            } else {
                dim3 grid((unsigned)((max_slice + 31) / 32), (unsigned)n_sums);
                launch(ex, splitk_sum_batch_kernel, grid, 256, 0, sums);
            }
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
    // blocks per job sized for the largest job (two 32 x 64 tiles per block), within 2 .. 592
    size_t bx = (max_job_elems + 4095) / 4096;
    if (bx < 2) bx = 2; if (bx > 592) bx = 592;
    dim3 grid((unsigned)bx, (unsigned)n_jobs);
    launch(ex, pack_weights_batch_kernel, grid, dim3(32, 8), 0, jobs_dev);
    ex.check("pack_weights_batch", bytes);
}
