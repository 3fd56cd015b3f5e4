// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <string>
#include <vector>
#include "../../include/revnet.h"

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------- context
struct ProfRec { const char *name; double bytes, flops; cudaEvent_t ev; };
struct StampRec { const char *name; double bytes, flops; int slot; };
constexpr int kStampSlots = 8192;
struct revnet_ctx {
    int device = 0;
    int sm_count = 148;
    std::string err;
    int *dev_status = nullptr;   // device word for bounded-wait time-outs
    unsigned int *counters = nullptr;   // zeroed words the kernels' grid-wide reductions count on (each leaves its word zero)
    int next_counter = 0;
    unsigned int *counter() { unsigned int *c = counters + next_counter; next_counter = (next_counter + 1) % kCounters; return c; }
    static constexpr int kCounters = 192;
    void *encode_tiled = nullptr; // driver entry point for tensor-map encoding
    cudaStream_t capture_stream = nullptr;   // private stream on which a train step is captured into a graph
    cudaStream_t side_stream = nullptr;      // weight gradients run here, beside the data-gradient chain
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaStream_t recon_stream = nullptr;     // a train step recomputes F here while the gradient steps of G run on the main stream
    cudaEvent_t ev_rfork = nullptr, ev_rjoin = nullptr;
    // per-kernel timing (revnet_profile_*): one event after every launch while enabled
    bool profiling = false;
    bool prof_detail = false;   // summary lines per launch shape, not only per kernel name
    std::vector<ProfRec> prof;
    std::vector<cudaEvent_t> ev_pool;
    size_t ev_used = 0;
    cudaEvent_t next_event();
    // device-side timeline (revnet_profile_enable(ctx, 3)): the stamped kernels write the %globaltimer of their first
    // CTA's start and their last CTA's end into a slot of their own; no events, no change to streams or graph replay
    bool stamping = false;
    unsigned long long *stamps = nullptr;      // [2][kStampSlots]: starts (minimum over CTAs), ends (maximum)
    int stamp_next = 0;
    std::vector<StampRec> stamp_recs;
};

// Function attributes (the dynamic shared-memory limit) belong to a device, not to the process: each kernel's
// launcher keeps one of these and sets its attributes the first time it runs on a device.  Setting them twice
// is harmless, so no lock: two threads that race both set the same value.
struct OncePerDevice {
    bool done[64] = {};
    bool first(int device) {
        if (device < 0 || device >= 64) return true;
        if (done[device]) return false;
        done[device] = true;
        return true;
    }
};

// A tensor of C = c0 + c1 channels stored as two NHWC tensors: channels [0,c0) in p0 (row
// stride c0) and [c0,c0+c1) in p1 (row stride c1).  c1 == 0: one plain tensor.
// q == 0: elements are float.  q > 0: elements are int32 fixed point, value = i * q with
// q = 2^-frac_bits (the exactly invertible coupling state of Section 3.2, "Numerical error").
struct Pair {
    float *p0;
    float *p1;
    int c0, c1;
    float q;
    __host__ __device__ int C() const { return c0 + c1; }
    __device__ __forceinline__ float *at(size_t row, int ch) const {
        return ch < c0 ? p0 + row * c0 + ch : p1 + row * c1 + (ch - c0);
    }
#ifdef __CUDACC__
    __device__ __forceinline__ float4 ld4(size_t row, int ch) const {
        const float *p = at(row, ch);
        return from_raw(*reinterpret_cast<const float4 *>(p));
    }
    // the 16 bytes as they are stored, and their values: split so that a streaming kernel can issue the loads of several
    // rows before it converts any of them (branch-free: the conversion instruction, not the adder route above)
    __device__ __forceinline__ float4 ld4_raw(size_t row, int ch) const { return *reinterpret_cast<const float4 *>(at(row, ch)); }
    __device__ __forceinline__ float4 from_raw(float4 r) const {
        if (q == 0.f) return r;
        return make_float4(__int2float_rn(__float_as_int(r.x)) * q, __int2float_rn(__float_as_int(r.y)) * q,
                           __int2float_rn(__float_as_int(r.z)) * q, __int2float_rn(__float_as_int(r.w)) * q);
    }
    // out = partner + sign * v on the stored representation (sign 0: out = v)
    __device__ __forceinline__ void couple(size_t row, int ch, float v, const Pair &partner, int sign) const {
        float *o = at(row, ch);
        if (q == 0.f) {
            if (sign) { float p = *partner.at(row, ch); v = sign > 0 ? p + v : p - v; }
            *o = v;
        } else {
            int iv = __float2int_rn(v * (1.f / q));
            if (sign) { int p = *reinterpret_cast<const int *>(partner.at(row, ch)); iv = sign > 0 ? p + iv : p - iv; }
            *reinterpret_cast<int *>(o) = iv;
        }
    }
    // store v in the tensor's format; returns the values as stored (dequantised)
    __device__ __forceinline__ float4 store4(size_t row, int ch, float4 v) const {
        float *o = at(row, ch);
        if (q == 0.f) { *reinterpret_cast<float4 *>(o) = v; return v; }
        const float s = 1.f / q;
        int4 iv = make_int4(__float2int_rn(v.x * s), __float2int_rn(v.y * s), __float2int_rn(v.z * s), __float2int_rn(v.w * s));
        *reinterpret_cast<int4 *>(o) = iv;
        return make_float4(__int2float_rn(iv.x) * q, __int2float_rn(iv.y) * q, __int2float_rn(iv.z) * q, __int2float_rn(iv.w) * q);
    }
    // out = partner + sign * v with the partner's 16 raw bytes already loaded; returns the stored values (dequantised)
    __device__ __forceinline__ float4 couple4_with(size_t row, int ch, float4 v, float4 praw, int sign) const {
        float *o = at(row, ch);
        if (q == 0.f) {
            if (sign > 0) { v.x = praw.x + v.x; v.y = praw.y + v.y; v.z = praw.z + v.z; v.w = praw.w + v.w; }
            else { v.x = praw.x - v.x; v.y = praw.y - v.y; v.z = praw.z - v.z; v.w = praw.w - v.w; }
            *reinterpret_cast<float4 *>(o) = v;
            return v;
        }
        const float s = 1.f / q;
        int4 iv = make_int4(__float2int_rn(v.x * s), __float2int_rn(v.y * s), __float2int_rn(v.z * s), __float2int_rn(v.w * s));
        const int4 p = make_int4(__float_as_int(praw.x), __float_as_int(praw.y), __float_as_int(praw.z), __float_as_int(praw.w));
        if (sign > 0) { iv.x = p.x + iv.x; iv.y = p.y + iv.y; iv.z = p.z + iv.z; iv.w = p.w + iv.w; }
        else { iv.x = p.x - iv.x; iv.y = p.y - iv.y; iv.z = p.z - iv.z; iv.w = p.w - iv.w; }
        *reinterpret_cast<int4 *>(o) = iv;
        return make_float4(__int2float_rn(iv.x) * q, __int2float_rn(iv.y) * q, __int2float_rn(iv.z) * q, __int2float_rn(iv.w) * q);
    }
    // four consecutive channels at once (ch % 4 == 0)
    __device__ __forceinline__ void couple4(size_t row, int ch, float4 v, const Pair &partner, int sign) const {
        float *o = at(row, ch);
        if (q == 0.f) {
            if (sign) {
                float4 p = *reinterpret_cast<const float4 *>(partner.at(row, ch));
                if (sign > 0) { v.x = p.x + v.x; v.y = p.y + v.y; v.z = p.z + v.z; v.w = p.w + v.w; }
                else { v.x = p.x - v.x; v.y = p.y - v.y; v.z = p.z - v.z; v.w = p.w - v.w; }
            }
            *reinterpret_cast<float4 *>(o) = v;
        } else {
            const float s = 1.f / q;
            int4 iv = make_int4(__float2int_rn(v.x * s), __float2int_rn(v.y * s), __float2int_rn(v.z * s), __float2int_rn(v.w * s));
            if (sign) {
                int4 p = *reinterpret_cast<const int4 *>(partner.at(row, ch));
                if (sign > 0) { iv.x = p.x + iv.x; iv.y = p.y + iv.y; iv.z = p.z + iv.z; iv.w = p.w + iv.w; }
                else { iv.x = p.x - iv.x; iv.y = p.y - iv.y; iv.z = p.z - iv.z; iv.w = p.w - iv.w; }
            }
            *reinterpret_cast<int4 *>(o) = iv;
        }
    }
#endif
};
static inline Pair single(float *p, int C, float q = 0.f) { return Pair{p, nullptr, C, 0, q}; }
static inline Pair halves(float *a, float *b, int c, float q = 0.f) { return Pair{a, b, c, c, q}; }

// Bump allocator over the caller's workspace; in dry mode it only measures.
struct Arena {
    char *base = nullptr;
    size_t off = 0, cap = 0, peak = 0;
    size_t high = 0;       // highest offset reached since the caller last set it (see block_backward)
    bool dry = true;
    bool overflow = false;
    void *alloc(size_t bytes) {
        size_t a = (off + 255) & ~size_t(255);
        off = a + bytes;
        if (off > peak) peak = off;
        if (off > high) high = off;
        if (!dry && off > cap) { overflow = true; return nullptr; }
        return dry ? (void *)(uintptr_t)(0x1000 + a) : base + a;   // non-null fake address in dry mode
    }
    template <class T> T *get(size_t n) { return (T *)alloc(n * sizeof(T)); }
    size_t mark() const { return off; }
    void release(size_t m) { off = m; }
};

// Everything a kernel launcher needs.
struct Exec {
    revnet_ctx *ctx = nullptr;
    cudaStream_t stream = nullptr;
    Arena ws;
    bool dry = true;       // true: size the workspace and count work, launch nothing
    int mode = 0;          // 0 bf16 tensor-core operands, 1 strict fp32
    float eps = 1e-5f;
    float q = 0.f;         // coupling-state format: 0 = float, else int32 fixed point with step q
    uint64_t flops = 0;    // dense conv/FC flops issued
    uint64_t launches = 0;
    bool failed = false;
    bool pdl = true;       // launch kernels with programmatic stream serialization (see launch())
    bool use_side = true;  // run weight gradients on the context's side stream (never while profiling)
    unsigned long long hold_ns = 0;   // profiling: the first mark() holds the stream this long so that launches queue up
    // called after every launch: error check, launch count and (when profiling) an event;
    // bytes / flops are the algorithmic traffic and work of that launch
    void check(const char *what, double bytes = 0, double flops = 0);
    void mark(const char *what);   // profiling boundary that is not a kernel (copies, step start)
    // timeline mode: the slot (start word; the end word is kStampSlots further on) the kernel about to be launched
    // stamps, or nullptr; the check() that follows the launch files the record
    unsigned long long *stamp_slot();
    int pending_slot = -1;
};

// Every kernel of the library is launched through here.  With ex.pdl the launch carries the
// programmatic-stream-serialization attribute: the grid may be scheduled while its predecessor in
// the stream still runs, and executes its set-up (barrier initialisation, tensor-memory
// allocation, index tables) meanwhile; each kernel calls pdl_enter() before it touches anything a
// predecessor wrote, which waits for the predecessor to complete and only then lets its own
// successor be scheduled, so at most two kernels of a stream overlap and ordering stays transitive.
template <class... KArgs, class... Args>
inline void launch(Exec &ex, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = ex.stream;
    cudaLaunchAttribute attr = {};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr; cfg.numAttrs = ex.pdl ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
// The same for a kernel that runs as clusters of `cluster_x` CTAs along x (grid.x a multiple of it).
template <class... KArgs, class... Args>
inline void launch_cluster(Exec &ex, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, int cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = ex.stream;
    cudaLaunchAttribute attr[2] = {};
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster_x; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = ex.pdl ? 2 : 1;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#ifdef __CUDACC__
// timeline stamps (see revnet_ctx::stamping): one thread per CTA, a few atomics per launch, nothing when s is null
__device__ __forceinline__ void stamp_begin(unsigned long long *s) {
    if (s && threadIdx.x == 0 && threadIdx.y == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        atomicMin(s, t);
    }
}
__device__ __forceinline__ void stamp_end(unsigned long long *s) {
    if (s && threadIdx.x == 0 && threadIdx.y == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        atomicMax(s + kStampSlots, t);
    }
}
// wait until the kernel before this one in the stream has completed (its writes are visible), then
// allow the kernel after this one to be scheduled
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

// One BN -> ReLU -> conv layer with its parameter and gradient pointers.
struct Layer {
    int cin = 0, cout = 0, k = 1, stride = 1;
    const float *W = nullptr, *gamma = nullptr, *beta = nullptr;
    float *dW = nullptr, *dgamma = nullptr, *dbeta = nullptr;
    const bf16 *Wp_fprop = nullptr;   // bf16 [cout][k][k][cin_pad]           (mode 0)
    const bf16 *Wp_dgrad = nullptr;   // bf16 [cin][k][k][cout_pad], taps mirrored (mode 0)
};

// Batch statistics of one tensor: per-channel mean and 1/sqrt(var + eps), [C] each (device).
// `valid` is host-side bookkeeping: whether a kernel enqueued earlier fills them.
// A fused convolution may leave them `pending`: its CTAs have written their partial sums (records of
// 2C floats, `parts` of them, in `part`) and the next kernel that normalises with them adds the
// records itself, in a fixed order, while its first tile is on the way -- cheaper than a grid-wide
// count and a reduction by the last CTA at the end of the producer.  That consumer also stores mean
// and rstd; anything else that wants them calls mom_finalize() first.
struct Moments {
    float *mean = nullptr, *rstd = nullptr;
    bool valid = false;
    float *part = nullptr;         // room for partial records (null: the producer must reduce itself)
    size_t part_cap = 0;           // floats
    int parts = 0;
    double inv_count = 0;          // 1 / pixels summed
    bool pending = false;
};
// One BN as its consumers see it: scale = gamma*rstd, shift = beta - mean*scale are derived on the
// fly, always with the same two roundings, so that the ReLU mask of the backward equals the forward's.
struct BnRef {
    const float *gamma, *beta, *mean, *rstd;
    // pending statistics (see Moments): the consumer reduces `parts` records of 2C floats and stores mean / rstd
    const float *part = nullptr;
    int parts = 0;
    double inv_count = 0;
    float eps = 0.f;
};
inline BnRef bn_ref(const float *gamma, const float *beta, const Moments &m, float eps) {
    BnRef b{gamma, beta, m.mean, m.rstd};
    if (m.pending) { b.part = m.part; b.parts = m.parts; b.inv_count = m.inv_count; b.eps = eps; }
    return b;
}
#ifdef __CUDACC__
__device__ __forceinline__ void bn_sc_sh(float g, float b, float mu, float r, float &sc, float &sh) {
    sc = __fmul_rn(g, r);
    sh = __fmaf_rn(-mu, sc, b);
}
__device__ __forceinline__ void bn_coef4(const BnRef &bn, int c, float4 &sc, float4 &sh, float4 &mu, float4 &rs) {
    const float4 g = *reinterpret_cast<const float4 *>(bn.gamma + c), b = *reinterpret_cast<const float4 *>(bn.beta + c);
    mu = *reinterpret_cast<const float4 *>(bn.mean + c); rs = *reinterpret_cast<const float4 *>(bn.rstd + c);
    bn_sc_sh(g.x, b.x, mu.x, rs.x, sc.x, sh.x); bn_sc_sh(g.y, b.y, mu.y, rs.y, sc.y, sh.y);
    bn_sc_sh(g.z, b.z, mu.z, rs.z, sc.z, sh.z); bn_sc_sh(g.w, b.w, mu.w, rs.w, sc.w, sh.w);
}
#endif

struct Geom { int N, H, W; size_t P() const { return (size_t)N * H * W; } };

// ---------------------------------------------------------------- elementwise.cu
Moments mom_alloc(Exec &ex, int C, bool with_part = false);
// pending statistics -> mean / rstd (one small kernel); no-op otherwise
void mom_finalize(Exec &ex, Moments &m, int C);
// batch statistics of t ([P,C]) -> mean, rstd (two kernels; the convolution epilogues produce the
// same quantities for the tensors they write)
void bn_stats(Exec &ex, Pair t, size_t P, Moments m);
// a = relu(scale*t + shift) written as one [P,C] tensor of float (strict) or bf16
void bn_relu_apply(Exec &ex, Pair t, size_t P, BnRef bn, void *a, bool a_bf16);
// BN+ReLU backward: da [P,C] fp32; t the BN input.  Unless sums_done (a data-gradient epilogue
// already wrote dgamma, dbeta and coef) the two reductions run first.  Then
//   out = dt                  (out_single: float or bf16 [P,C])   when out_pair.p0 == nullptr
//   out_pair = add + dt       (fp32 pair; add.p0 == nullptr: plain dt), optionally also
//   out_cast = bf16 copy of out_pair as one [P,C] tensor (the next function's upstream operand)
void bn_relu_bwd(Exec &ex, const float *da, Pair t, size_t P, BnRef bn, float *dgamma, float *dbeta, float *coef,
                 bool sums_done, void *out_single, bool out_bf16, Pair add, Pair out_pair, bf16 *out_cast);
// copy a pair into one [P,C] tensor of float or bf16
void concat_cast(Exec &ex, Pair src, size_t P, void *dst, bool dst_bf16);
void maxpool_fwd(Exec &ex, const float *in, float *out, int N, int H, int W, int C);
void maxpool_bwd(Exec &ex, const float *in, const float *dout, float *din, int N, int H, int W, int C);
void head_fwd(Exec &ex, Pair y, int N, int HW, const float *Wfc, const float *bfc, const int32_t *labels,
              int n_classes, float *feat, float *logits, float *dlogits, float *loss, int32_t *pred);
void head_bwd(Exec &ex, Pair dy, int N, int HW, const float *Wfc, const float *feat, const float *dlogits,
              int n_classes, float *dWfc, float *dbfc, float *dfeat);
void sgd_update(Exec &ex, float *params, const float *grads, float *mom, size_t n,
                const uint32_t *seg_end, const uint8_t *seg_decay, int n_seg,
                float lr, float momentum, float wd, bool quad_aligned);   // quad_aligned: every segment but the last ends on a multiple of four
// max |a - b| over n elements of two state tensors (float, or fixed point when q > 0)
void max_abs_diff(Exec &ex, const float *a, const float *b, size_t n, float q, float *out /*1 float, pre-zeroed*/);
void fill_zero(Exec &ex, void *p, size_t bytes);
// shortcut of a down-sampling unit: S(x) = 2x2 average pool (stride 2) + zero channels up to cout, in the state format
// (q as in Pair); and its adjoint on float gradients (first cin channels, weight 1/4 per window position)
void shortcut_fwd(Exec &ex, const float *x, float *out, int N, int H, int W, int cin, int cout, float q);
void shortcut_bwd(Exec &ex, const float *d, float *gx, int N, int H, int W, int cin, int cout);
// out[n, 2i, 2j, :] = in[n, i, j, :], zero elsewhere; out is [N, 2Ho, 2Wo, C]
void upsample_zero_bf16(Exec &ex, const bf16 *in, bf16 *out, int N, int Ho, int Wo, int C);

// ---------------------------------------------------------------- conv_simt.cu
// Operand element type of the activated tensor / upstream gradient: float or bf16.
// out = partner + sign*conv(a)   (sign 0: out = conv(a), partner unused)
void conv_fprop_simt(Exec &ex, const void *a, bool a_bf16, Geom gi, const Layer &L, Pair out, Pair partner, int sign);
void conv_dgrad_simt(Exec &ex, const void *g, bool g_bf16, Geom gi, const Layer &L, float *da);
void conv_wgrad_simt(Exec &ex, const void *g, bool g_bf16, const void *a, bool a_bf16, Geom gi, const Layer &L, float *dW);

// ---------------------------------------------------------------- stem.cu
// the stem convolution of the image (few input channels), fp32; false: shape not taken, nothing launched
bool stem_fprop(Exec &ex, const float *img, Geom gi, const Layer &L, Pair out);
bool stem_wgrad(Exec &ex, const float *img, const float *gout, Geom gi, const Layer &L, float *dW);

// ---------------------------------------------------------------- conv_tc.cu
// What a data-gradient epilogue needs to fuse the two sums of the BN+ReLU backward of the layer's
// own BN: its input t, its coefficients, and where dgamma, dbeta and coef[3][C] go.
struct BnBwdReq { Pair t; BnRef bn; float *dgamma, *dbeta, *coef; };
// Reductions a convolution epilogue is asked to fuse.
struct EpiReq {
    Moments *stats = nullptr;          // statistics of the stored result
    const BnBwdReq *bnbwd = nullptr;   // data gradient: sums of the BN+ReLU backward
};
void *tc_encoder(revnet_ctx *ctx);     // cuTensorMapEncodeTiled, resolved once per context (nullptr if unavailable)
void tc_pack_now(Exec &ex, const float *W, bf16 *out, int cin, int cout, int k, bool transposed);
// bf16 weight packs of the tensor-core kernels, built once per train step
struct PackJob { const float *W; bf16 *out; int Co, Ci, k, rows_pad, cols_pad, transposed; };
size_t tc_pack_elems(int cin, int cout, int k, bool transposed);
PackJob tc_pack_job(const float *W, bf16 *out, int cin, int cout, int k, bool transposed);
void tc_pack_batch(Exec &ex, const PackJob *jobs_dev, int n_jobs, double bytes, size_t max_job_elems);

// ---------------------------------------------------------------- block.cu
struct FnSaved;   // activations kept from a residual function's (re)computation
// out = partner + sign * Fn(u); if saved != nullptr the per-layer tensors stay in the workspace
// skip_last_conv: only rebuild the saved tensors (used to re-derive a stored layer's operands)
// mom_in: statistics of u if a kernel enqueued earlier provides them (else they are computed here);
// mom_out: where the last convolution's epilogue should leave the statistics of `out`
// (mom_out->valid tells whether it did).
void fn_forward(Exec &ex, Geom g, Pair u, const Moments *mom_in, const std::vector<Layer> &layers, Pair partner, Pair out,
                int sign, Moments *mom_out, FnSaved *saved, bool skip_last_conv);
// dgin_out = add + (dFn/du)^T gup, parameter gradients written through the layers' pointers;
// gup_cast: bf16 [P,C] copy of gup if the caller already has one; dgin_cast: if non-null, a bf16
// [P,C] copy of dgin_out is written there as well
void fn_backward(Exec &ex, Geom g, Pair u, const std::vector<Layer> &layers, FnSaved &saved, Pair gup, const bf16 *gup_cast,
                 Pair add, Pair dgin_out, bf16 *dgin_cast);
struct FnSaved {
    std::vector<void *> a;        // activated input of each conv
    std::vector<float *> t;       // BN input of each layer beyond the first (conv outputs)
    std::vector<Moments> bn;
    Geom gin;
};
// Statistics hand-off between blocks of a stage (all optional, nullptr = compute where needed):
//   forward : mx2 = statistics of x2 (if valid); my1, my2: where those of y1, y2 are left
//   backward: m1 in = statistics of y1, out = statistics of x1; m2 out = statistics of x2;
//             m2_use: statistics F must use for x2 when the forward pass took them from elsewhere
//             (the first block of a stage), so that F is recomputed bit for bit;
//             m1_out: where the statistics of x1 go instead of m1 (default: m1 is overwritten)
//   overlap : the recomputation of F (x1 = y1 - F(x2)) runs on the context's reconstruction stream beside
//             the gradient steps of G, which still read y1 and its statistics: the caller must then pass
//             x1 != y1 and m1_out != m1
void block_forward(Exec &ex, Geom g, int c, const std::vector<Layer> &F, const std::vector<Layer> &G,
                   float *x1, float *x2, float *y1, float *y2,
                   const Moments *mx2 = nullptr, Moments *my1 = nullptr, Moments *my2 = nullptr);
void block_backward(Exec &ex, Geom g, int c, const std::vector<Layer> &F, const std::vector<Layer> &G,
                    const float *y1, const float *y2, const float *dy1, const float *dy2,
                    float *x1, float *x2, float *dx1, float *dx2,
                    Moments *m1 = nullptr, Moments *m2 = nullptr, const Moments *m2_use = nullptr,
                    const bf16 *dy2_cast = nullptr, bf16 *dx2_cast = nullptr, Moments *m1_out = nullptr, bool overlap = false);

static inline int conv_out(int in, int k, int s) { return (in + 2 * (k / 2) - k) / s + 1; }
