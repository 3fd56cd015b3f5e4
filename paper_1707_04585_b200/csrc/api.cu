// C ABI: context management and the block-level entry points.
#include "common.cuh"
#include "tc_ptx.cuh"
#include <string.h>
#include <stdio.h>
#include <math.h>
#include <atomic>
#include <algorithm>

static int fail(revnet_ctx *ctx, int code, const std::string &msg) { if (ctx) ctx->err = msg; return code; }

extern "C" int revnet_create(revnet_ctx **out, int device) {
    if (!out) return REVNET_E_INVALID_ARG;
    revnet_ctx *c = new revnet_ctx();
    c->device = device;
    if (device >= 0) {
        // device < 0 makes a planning-only context: sizes and layouts can be queried without a GPU
        int sm = 0;
        if (cudaSetDevice(device) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
            cudaMalloc(&c->dev_status, 1024) != cudaSuccess || cudaMemset(c->dev_status, 0, 1024) != cudaSuccess ||
            cudaMalloc(&c->stamps, 2 * kStampSlots * sizeof(unsigned long long)) != cudaSuccess ||
            cudaStreamCreateWithFlags(&c->capture_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&c->recon_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_rfork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_rjoin, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            delete c;
            return REVNET_E_CUDA;
        }
        c->sm_count = sm;
        c->counters = reinterpret_cast<unsigned int *>(c->dev_status) + 64;
    }
    *out = c;
    return REVNET_OK;
}

extern "C" int revnet_destroy(revnet_ctx *ctx) {
    if (!ctx) return REVNET_OK;
    for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    if (ctx->stamps) cudaFree(ctx->stamps);
    if (ctx->capture_stream) cudaStreamDestroy(ctx->capture_stream);
    if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
    if (ctx->recon_stream) cudaStreamDestroy(ctx->recon_stream);
    if (ctx->ev_rfork) cudaEventDestroy(ctx->ev_rfork);
    if (ctx->ev_rjoin) cudaEventDestroy(ctx->ev_rjoin);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    delete ctx;
    return REVNET_OK;
}

extern "C" const char *revnet_last_error(const revnet_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

static int check_fn(const revnet_fn_desc &f, int c) {
    if (f.n_layers < 1 || f.n_layers > 3) return 0;
    for (int l = 0; l < f.n_layers; l++) {
        if ((f.k[l] != 1 && f.k[l] != 3) || f.cin[l] < 4 || f.cin[l] % 4 || f.cout[l] < 4 || f.cout[l] % 4) return 0;
        if (l && f.cin[l] != f.cout[l - 1]) return 0;
    }
    return f.cin[0] == c && f.cout[f.n_layers - 1] == c;
}
static int check_desc(revnet_ctx *ctx, const revnet_block_desc *d) {
    if (!ctx || !d) return fail(ctx, REVNET_E_INVALID_ARG, "null descriptor");
    if (d->N < 1 || d->H < 1 || d->W < 1 || d->c < 4 || (d->mode != 0 && d->mode != 1) || d->state_frac_bits < 0 || d->state_frac_bits > 24)
        return fail(ctx, REVNET_E_INVALID_ARG, "block descriptor: N,H,W >= 1, c >= 4, mode in {0,1}, state_frac_bits in [0,24]");
    if (d->c % 4 || !check_fn(d->F, d->c) || !check_fn(d->G, d->c))
        return fail(ctx, REVNET_E_UNSUPPORTED_SHAPE, "block descriptor: channels must be multiples of 4, kernels 1 or 3, F and G must map c -> c");
    if ((size_t)d->N * d->H * d->W >= (1u << 30)) return fail(ctx, REVNET_E_UNSUPPORTED_SHAPE, "block descriptor: too many pixels");
    return REVNET_OK;
}

static std::vector<Layer> layers_of(const revnet_fn_desc &f, const revnet_fn_params *p, const revnet_fn_grads *g) {
    std::vector<Layer> v(f.n_layers);
    for (int l = 0; l < f.n_layers; l++) {
        v[l].cin = f.cin[l]; v[l].cout = f.cout[l]; v[l].k = f.k[l]; v[l].stride = 1;
        if (p) {
            v[l].W = p->W[l]; v[l].gamma = p->gamma[l]; v[l].beta = p->beta[l];
            v[l].Wp_fprop = (const bf16 *)p->Wpack_fprop[l]; v[l].Wp_dgrad = (const bf16 *)p->Wpack_dgrad[l];
        }
        if (g) { v[l].dW = g->dW[l]; v[l].dgamma = g->dgamma[l]; v[l].dbeta = g->dbeta[l]; }
    }
    return v;
}

static bool aligned16(std::initializer_list<const void *> ps) {
    for (const void *p : ps) if ((uintptr_t)p & 15) return false;
    return true;
}
static bool fn_ptrs_ok(const revnet_fn_desc &f, const revnet_fn_params *p, const revnet_fn_grads *g, bool need_g, bool *misaligned) {
    if (!p || (need_g && !g)) return false;
    for (int l = 0; l < f.n_layers; l++) {
        if (!p->W[l] || !p->gamma[l] || !p->beta[l]) return false;
        if (!aligned16({p->W[l], p->gamma[l], p->beta[l]})) *misaligned = true;
        if (need_g) {
            if (!g->dW[l] || !g->dgamma[l] || !g->dbeta[l]) return false;
            if (!aligned16({g->dW[l], g->dgamma[l], g->dbeta[l]})) *misaligned = true;
        }
    }
    return true;
}

extern "C" int revnet_block_workspace_bytes(revnet_ctx *ctx, const revnet_block_desc *d, size_t *fwd_bytes, size_t *bwd_bytes) {
    int rc = check_desc(ctx, d);
    if (rc) return rc;
    Geom g{d->N, d->H, d->W};
    float *fake = (float *)0x1000;
    for (int pass = 0; pass < 2; pass++) {
        Exec ex; ex.ctx = ctx; ex.dry = true; ex.ws.dry = true; ex.mode = d->mode; ex.eps = d->eps;
        auto F = layers_of(d->F, nullptr, nullptr), G = layers_of(d->G, nullptr, nullptr);
        if (pass == 0) block_forward(ex, g, d->c, F, G, fake, fake, fake, fake);
        else block_backward(ex, g, d->c, F, G, fake, fake, fake, fake, fake, fake, fake, fake);
        size_t *o = pass == 0 ? fwd_bytes : bwd_bytes;
        if (o) *o = ex.ws.peak + 256;
    }
    return REVNET_OK;
}

static int finish(revnet_ctx *ctx, Exec &ex, const char *who) {
    if (ex.ws.overflow) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, std::string(who) + ": workspace too small");
    if (ex.failed) return REVNET_E_CUDA;
    return REVNET_OK;
}

extern "C" int revnet_block_fwd(revnet_ctx *ctx, const revnet_block_desc *d, const void *x1, const void *x2,
                                const revnet_fn_params *Fp, const revnet_fn_params *Gp, void *y1, void *y2,
                                void *workspace, size_t workspace_bytes, void *stream) {
    int rc = check_desc(ctx, d);
    if (rc) return rc;
    bool mis = false;
    if (!x1 || !x2 || !y1 || !y2 || !workspace || !fn_ptrs_ok(d->F, Fp, nullptr, false, &mis) || !fn_ptrs_ok(d->G, Gp, nullptr, false, &mis))
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_block_fwd: null pointer");
    if (mis || !aligned16({x1, x2, y1, y2, workspace})) return fail(ctx, REVNET_E_MISALIGNED, "revnet_block_fwd: pointers must be 16-byte aligned");
    size_t need = 0;
    revnet_block_workspace_bytes(ctx, d, &need, nullptr);
    if (workspace_bytes < need) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_block_fwd: workspace too small");
    Exec ex; ex.ctx = ctx; ex.dry = false; ex.mode = d->mode; ex.eps = d->eps; ex.stream = (cudaStream_t)stream;
    ex.q = d->state_frac_bits ? ldexpf(1.f, -d->state_frac_bits) : 0.f;
    ex.ws.dry = false; ex.ws.base = (char *)workspace; ex.ws.cap = workspace_bytes;
    block_forward(ex, Geom{d->N, d->H, d->W}, d->c, layers_of(d->F, Fp, nullptr), layers_of(d->G, Gp, nullptr),
                  (float *)x1, (float *)x2, (float *)y1, (float *)y2);
    return finish(ctx, ex, "revnet_block_fwd");
}

extern "C" int revnet_block_bwd(revnet_ctx *ctx, const revnet_block_desc *d, const void *y1, const void *y2,
                                const float *dy1, const float *dy2, const revnet_fn_params *Fp, const revnet_fn_params *Gp,
                                void *x1, void *x2, float *dx1, float *dx2, const revnet_fn_grads *gF, const revnet_fn_grads *gG,
                                void *workspace, size_t workspace_bytes, void *stream) {
    int rc = check_desc(ctx, d);
    if (rc) return rc;
    bool mis = false;
    if (!y1 || !y2 || !dy1 || !dy2 || !x1 || !x2 || !dx1 || !dx2 || !workspace ||
        !fn_ptrs_ok(d->F, Fp, gF, true, &mis) || !fn_ptrs_ok(d->G, Gp, gG, true, &mis))
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_block_bwd: null pointer");
    if (mis || !aligned16({y1, y2, dy1, dy2, x1, x2, dx1, dx2, workspace}))
        return fail(ctx, REVNET_E_MISALIGNED, "revnet_block_bwd: pointers must be 16-byte aligned");
    size_t need = 0;
    revnet_block_workspace_bytes(ctx, d, nullptr, &need);
    if (workspace_bytes < need) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_block_bwd: workspace too small");
    Exec ex; ex.ctx = ctx; ex.dry = false; ex.mode = d->mode; ex.eps = d->eps; ex.stream = (cudaStream_t)stream;
    ex.q = d->state_frac_bits ? ldexpf(1.f, -d->state_frac_bits) : 0.f;
    ex.ws.dry = false; ex.ws.base = (char *)workspace; ex.ws.cap = workspace_bytes;
    block_backward(ex, Geom{d->N, d->H, d->W}, d->c, layers_of(d->F, Fp, gF), layers_of(d->G, Gp, gG),
                   (const float *)y1, (const float *)y2, dy1, dy2, (float *)x1, (float *)x2, dx1, dx2);
    return finish(ctx, ex, "revnet_block_bwd");
}

// ---- bf16 weight packs made once and handed to the block calls (a train step makes its own, once per step)
static bool packable(const revnet_block_desc *d, const revnet_fn_desc &f, int l) {
    return d->mode == 0 && f.cin[l] % 8 == 0 && f.cout[l] % 8 == 0;
}
static size_t pack_bytes_of(const revnet_block_desc *d) {
    size_t total = 0;
    for (const revnet_fn_desc *f : {&d->F, &d->G})
        for (int l = 0; l < f->n_layers; l++)
            if (packable(d, *f, l))
                for (int tr = 0; tr < 2; tr++) total += (tc_pack_elems(f->cin[l], f->cout[l], f->k[l], tr != 0) * sizeof(bf16) + 255) & ~size_t(255);
    return total;
}
extern "C" int revnet_block_pack_bytes(revnet_ctx *ctx, const revnet_block_desc *d, size_t *bytes) {
    int rc = check_desc(ctx, d);
    if (rc) return rc;
    if (!bytes) return fail(ctx, REVNET_E_INVALID_ARG, "revnet_block_pack_bytes: null pointer");
    *bytes = pack_bytes_of(d);
    return REVNET_OK;
}
extern "C" int revnet_pack_weights(revnet_ctx *ctx, const revnet_block_desc *d, revnet_fn_params *Fp, revnet_fn_params *Gp,
                                   void *pack_buffer, size_t pack_bytes, void *stream) {
    int rc = check_desc(ctx, d);
    if (rc) return rc;
    bool mis = false;
    if (!fn_ptrs_ok(d->F, Fp, nullptr, false, &mis) || !fn_ptrs_ok(d->G, Gp, nullptr, false, &mis))
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_pack_weights: null pointer");
    const size_t need = pack_bytes_of(d);
    if (need && !pack_buffer) return fail(ctx, REVNET_E_INVALID_ARG, "revnet_pack_weights: null pack buffer");
    if (mis || ((uintptr_t)pack_buffer & 255)) return fail(ctx, REVNET_E_MISALIGNED, "revnet_pack_weights: the pack buffer must be 256-byte aligned, parameters 16-byte aligned");
    if (pack_bytes < need) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_pack_weights: pack buffer holds " + std::to_string(pack_bytes) + " bytes, " + std::to_string(need) + " needed");
    Exec ex; ex.ctx = ctx; ex.dry = false; ex.mode = d->mode; ex.eps = d->eps; ex.stream = (cudaStream_t)stream;
    char *at = (char *)pack_buffer;
    revnet_fn_params *ps[2] = {Fp, Gp};
    const revnet_fn_desc *fs[2] = {&d->F, &d->G};
    for (int i = 0; i < 2; i++)
        for (int l = 0; l < 3; l++) {
            ps[i]->Wpack_fprop[l] = ps[i]->Wpack_dgrad[l] = nullptr;
            if (l >= fs[i]->n_layers || !packable(d, *fs[i], l)) continue;
            for (int tr = 0; tr < 2; tr++) {
                tc_pack_now(ex, ps[i]->W[l], (bf16 *)at, fs[i]->cin[l], fs[i]->cout[l], fs[i]->k[l], tr != 0);
                (tr ? ps[i]->Wpack_dgrad[l] : ps[i]->Wpack_fprop[l]) = at;
                at += (tc_pack_elems(fs[i]->cin[l], fs[i]->cout[l], fs[i]->k[l], tr != 0) * sizeof(bf16) + 255) & ~size_t(255);
            }
        }
    return finish(ctx, ex, "revnet_pack_weights");
}

// ---- block forward on the library's own static scratch: for callers that cannot allocate
// Some integrations run where device allocation is off the table: inside a memory pool whose owner
// forbids side allocations, in a real-time or safety-checked loop that must not touch the
// allocator, or in a plugin that is handed tensors but no allocator.  For them this variant of
// revnet_block_fwd takes its scratch from a fixed array that lives in the library image.
#define REVNET_NOALLOC_SCRATCH_BYTES (16u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[REVNET_NOALLOC_SCRATCH_BYTES];
// device address of the array, looked up once per device (the array's name is only a host-side
// handle in host code and must never be handed to a kernel as if it were a pointer)
static std::atomic<void *> g_noalloc_ptr[64];

extern "C" int revnet_block_fwd_noalloc(revnet_ctx *ctx, const revnet_block_desc *d, const void *x1, const void *x2,
                                        const revnet_fn_params *Fp, const revnet_fn_params *Gp, void *y1, void *y2, void *stream) {
    int rc = check_desc(ctx, d);
    if (rc) return rc;
    bool mis = false;
    if (!x1 || !x2 || !y1 || !y2 || !fn_ptrs_ok(d->F, Fp, nullptr, false, &mis) || !fn_ptrs_ok(d->G, Gp, nullptr, false, &mis))
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_block_fwd_noalloc: null pointer");
    if (mis || !aligned16({x1, x2, y1, y2})) return fail(ctx, REVNET_E_MISALIGNED, "revnet_block_fwd_noalloc: pointers must be 16-byte aligned");
    size_t need = 0;
    revnet_block_workspace_bytes(ctx, d, &need, nullptr);
    if (need > REVNET_NOALLOC_SCRATCH_BYTES)
        return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_block_fwd_noalloc: this shape needs " + std::to_string(need) +
                    " bytes of scratch, the static array holds " + std::to_string((size_t)REVNET_NOALLOC_SCRATCH_BYTES) +
                    "; use revnet_block_fwd with a caller workspace");
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return fail(ctx, REVNET_E_CUDA, "revnet_block_fwd_noalloc: no current device");
    if (dev != ctx->device) return fail(ctx, REVNET_E_INVALID_ARG, "revnet_block_fwd_noalloc: the context's device must be current");
    void *scratch = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        // one-time set-up for this device (with it current): resolve the array's device address.  Two threads that
        // race here both get the same address from the runtime.
        cudaError_t e = cudaGetSymbolAddress(&scratch, g_noalloc_scratch);
        if (e != cudaSuccess || !scratch)
            return fail(ctx, REVNET_E_CUDA, std::string("revnet_block_fwd_noalloc: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
        g_noalloc_ptr[dev].store(scratch, std::memory_order_release);
    }
    Exec ex; ex.ctx = ctx; ex.dry = false; ex.mode = d->mode; ex.eps = d->eps; ex.stream = (cudaStream_t)stream;
    ex.q = d->state_frac_bits ? ldexpf(1.f, -d->state_frac_bits) : 0.f;
    ex.ws.dry = false; ex.ws.base = (char *)scratch; ex.ws.cap = REVNET_NOALLOC_SCRATCH_BYTES;
    // nothing in the block forward relies on zeroed scratch: every region is written before it is read
    block_forward(ex, Geom{d->N, d->H, d->W}, d->c, layers_of(d->F, Fp, nullptr), layers_of(d->G, Gp, nullptr),
                  (float *)x1, (float *)x2, (float *)y1, (float *)y2);
    return finish(ctx, ex, "revnet_block_fwd_noalloc");
}

// ---- stored (non-reversible) BN -> ReLU -> conv layer: forward keeps nothing, backward rebuilds its
// operands from the stored input (Section 3.2: inputs of non-reversible layers are kept)
static int check_trans(revnet_ctx *ctx, const revnet_transition_desc *d) {
    if (!ctx || !d) return fail(ctx, REVNET_E_INVALID_ARG, "null descriptor");
    if (d->N < 1 || d->H < 1 || d->W < 1 || (d->mode != 0 && d->mode != 1) || d->state_frac_bits < 0 || d->state_frac_bits > 24 ||
        (d->in_split != 0 && d->in_split != 1))
        return fail(ctx, REVNET_E_INVALID_ARG, "transition descriptor: bad N/H/W/mode/state_frac_bits/in_split");
    if ((d->k != 1 && d->k != 3) || (d->stride != 1 && d->stride != 2) || d->cin < 4 || d->cin % (d->in_split ? 8 : 4) || d->cout < 8 || d->cout % 8)
        return fail(ctx, REVNET_E_UNSUPPORTED_SHAPE, "transition descriptor: k in {1,3}, stride in {1,2}, cin % 4 (8 when split), cout % 8");
    return REVNET_OK;
}
static void trans_run(Exec &ex, const revnet_transition_desc *d, bool backward, const void *in1, const void *in2,
                      const float *W, const float *gamma, const float *beta, void *out1, void *out2,
                      const float *dout1, const float *dout2, float *din1, float *din2, float *dW, float *dgamma, float *dbeta) {
    const float q = ex.q;
    Layer L; L.cin = d->cin; L.cout = d->cout; L.k = d->k; L.stride = d->stride;
    L.W = W; L.gamma = gamma; L.beta = beta; L.dW = dW; L.dgamma = dgamma; L.dbeta = dbeta;
    std::vector<Layer> T{L};
    Geom g{d->N, d->H, d->W};
    Pair tin = d->in_split ? halves((float *)in1, (float *)in2, d->cin / 2, q) : single((float *)in1, d->cin);
    const int ch = d->cout / 2;
    if (!backward) {
        fn_forward(ex, g, tin, nullptr, T, Pair{}, halves((float *)out1, (float *)out2, ch, q), 0, nullptr, nullptr, false);
    } else {
        FnSaved sv;
        size_t m = ex.ws.mark();
        fn_forward(ex, g, tin, nullptr, T, Pair{}, Pair{}, 0, nullptr, &sv, true);
        Pair gout = d->in_split ? halves(din1, din2, d->cin / 2) : single(din1, d->cin);
        fn_backward(ex, g, tin, T, sv, halves((float *)dout1, (float *)dout2, ch), nullptr, Pair{}, gout, nullptr);
        ex.ws.release(m);
    }
}
static Exec trans_exec(revnet_ctx *ctx, const revnet_transition_desc *d, bool dry, void *ws, size_t ws_bytes, void *stream) {
    Exec ex; ex.ctx = ctx; ex.dry = dry; ex.ws.dry = dry; ex.mode = d->mode; ex.eps = d->eps; ex.stream = (cudaStream_t)stream;
    ex.q = d->state_frac_bits ? ldexpf(1.f, -d->state_frac_bits) : 0.f;
    ex.ws.base = (char *)ws; ex.ws.cap = ws_bytes;
    return ex;
}
extern "C" int revnet_transition_workspace_bytes(revnet_ctx *ctx, const revnet_transition_desc *d, size_t *fwd_bytes, size_t *bwd_bytes) {
    int rc = check_trans(ctx, d);
    if (rc) return rc;
    float *f = (float *)0x1000;
    for (int pass = 0; pass < 2; pass++) {
        Exec ex = trans_exec(ctx, d, true, nullptr, 0, nullptr);
        trans_run(ex, d, pass == 1, f, f, f, f, f, f, f, f, f, f, f, f, f, f);
        size_t *o = pass == 0 ? fwd_bytes : bwd_bytes;
        if (o) *o = ex.ws.peak + 256;
    }
    return REVNET_OK;
}
extern "C" int revnet_transition_fwd(revnet_ctx *ctx, const revnet_transition_desc *d, const void *in1, const void *in2,
                                     const float *W, const float *gamma, const float *beta, void *out1, void *out2,
                                     void *workspace, size_t workspace_bytes, void *stream) {
    int rc = check_trans(ctx, d);
    if (rc) return rc;
    if (!in1 || (d->in_split && !in2) || !W || !gamma || !beta || !out1 || !out2 || !workspace)
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_transition_fwd: null pointer");
    if (!aligned16({in1, in2, W, gamma, beta, out1, out2, workspace})) return fail(ctx, REVNET_E_MISALIGNED, "revnet_transition_fwd: pointers must be 16-byte aligned");
    size_t need = 0;
    revnet_transition_workspace_bytes(ctx, d, &need, nullptr);
    if (workspace_bytes < need) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_transition_fwd: workspace too small");
    Exec ex = trans_exec(ctx, d, false, workspace, workspace_bytes, stream);
    trans_run(ex, d, false, in1, in2, W, gamma, beta, out1, out2, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr);
    return finish(ctx, ex, "revnet_transition_fwd");
}
extern "C" int revnet_transition_bwd(revnet_ctx *ctx, const revnet_transition_desc *d, const void *in1, const void *in2,
                                     const float *dout1, const float *dout2, const float *W, const float *gamma, const float *beta,
                                     float *din1, float *din2, float *dW, float *dgamma, float *dbeta,
                                     void *workspace, size_t workspace_bytes, void *stream) {
    int rc = check_trans(ctx, d);
    if (rc) return rc;
    if (!in1 || (d->in_split && (!in2 || !din2)) || !dout1 || !dout2 || !W || !gamma || !beta || !din1 || !dW || !dgamma || !dbeta || !workspace)
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_transition_bwd: null pointer");
    if (!aligned16({in1, in2, dout1, dout2, W, gamma, beta, din1, din2, dW, dgamma, dbeta, workspace}))
        return fail(ctx, REVNET_E_MISALIGNED, "revnet_transition_bwd: pointers must be 16-byte aligned");
    size_t need = 0;
    revnet_transition_workspace_bytes(ctx, d, nullptr, &need);
    if (workspace_bytes < need) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_transition_bwd: workspace too small");
    Exec ex = trans_exec(ctx, d, false, workspace, workspace_bytes, stream);
    trans_run(ex, d, true, in1, in2, W, gamma, beta, nullptr, nullptr, dout1, dout2, din1, din2, dW, dgamma, dbeta);
    return finish(ctx, ex, "revnet_transition_bwd");
}

// ---- device-side status
extern "C" int revnet_check_device(revnet_ctx *ctx, void *stream) {
    if (!ctx) return REVNET_E_INVALID_ARG;
    if (!ctx->dev_status) return REVNET_OK;
    int st = 0;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&st, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return fail(ctx, REVNET_E_CUDA, std::string("revnet_check_device: ") + cudaGetErrorString(cudaGetLastError()));
    if (st != 0) {
        // a kernel that gave up never counted itself out of its grid-wide reduction: zero the counter words as well,
        // or a later kernel handed the same word would elect its last CTA too early
        cudaMemsetAsync(ctx->dev_status, 0, 1024, s);
        cudaStreamSynchronize(s);
        return fail(ctx, st, "a kernel gave up a bounded wait (device status " + std::to_string(st) + ")");
    }
    return REVNET_OK;
}

// One CTA waits, with the caller's limit, on a shared-memory barrier that nothing arrives on: the wait runs out,
// the kernel records the status and returns normally -- the path every bounded wait in the library takes on expiry.
__global__ void selftest_wait_kernel(unsigned long long limit_ns, int *status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!tc::mbar_wait(&bar, 0, limit_ns)) atomicExch(status, (int)REVNET_E_TIMEOUT);
    }
}
extern "C" int revnet_selftest_bounded_wait(revnet_ctx *ctx, uint64_t limit_ns, void *stream) {
    if (!ctx || !ctx->dev_status) return REVNET_E_INVALID_ARG;
    if (limit_ns == 0 || limit_ns > 100000000ull) return fail(ctx, REVNET_E_INVALID_ARG, "revnet_selftest_bounded_wait: limit must be in (0, 100 ms]");
    selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((unsigned long long)limit_ns, ctx->dev_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, REVNET_E_CUDA, std::string("revnet_selftest_bounded_wait: ") + cudaGetErrorString(e));
    return REVNET_OK;
}

// ---- per-kernel timing
extern "C" int revnet_profile_enable(revnet_ctx *ctx, int on) {
    if (!ctx) return REVNET_E_INVALID_ARG;
    ctx->profiling = on == 1 || on == 2;
    ctx->prof_detail = on == 2;
    ctx->stamping = on == 3;
    ctx->prof.clear();
    ctx->ev_used = 0;
    ctx->stamp_recs.clear();
    ctx->stamp_next = 0;
    return REVNET_OK;
}

extern "C" int revnet_profile_summary(revnet_ctx *ctx, char *buf, size_t buflen, size_t *needed) {
    if (!ctx || (!buf && buflen)) return REVNET_E_INVALID_ARG;
    struct Acc { std::string name; uint64_t n = 0; double ms = 0, bytes = 0, flops = 0; };
    std::vector<Acc> acc;
    if (ctx->stamping) {
        // timeline mode: the stamps of the last step that ran (the caller has synchronised, or we do)
        std::vector<unsigned long long> h(2 * kStampSlots);
        if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(h.data(), ctx->stamps, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess)
            return fail(ctx, REVNET_E_CUDA, std::string("revnet_profile_summary: ") + cudaGetErrorString(cudaGetLastError()));
        std::vector<std::pair<unsigned long long, unsigned long long>> iv;
        for (const StampRec &r : ctx->stamp_recs) {
            const unsigned long long t0 = h[r.slot], t1 = h[kStampSlots + r.slot];
            if (t1 == 0 || t0 == ~0ull || t1 < t0) continue;      // the kernel did not run in the last step
            char key[160];
            snprintf(key, sizeof key, "%s|%.0f|%.0f", r.name, r.bytes, r.flops);
            Acc *a = nullptr;
            for (auto &x : acc) if (x.name == key) { a = &x; break; }
            if (!a) { acc.push_back(Acc()); a = &acc.back(); a->name = key; }
            a->n++; a->ms += (double)(t1 - t0) * 1e-6; a->bytes += r.bytes; a->flops += r.flops;
            iv.push_back({t0, t1});
        }
        // time during which at least one stamped kernel ran, and the span from the first start to the last end
        std::sort(iv.begin(), iv.end());
        double busy = 0; unsigned long long lo = 0, hi = 0;
        for (auto &p : iv) {
            if (hi == 0) { lo = p.first; hi = p.second; }
            else if (p.first <= hi) { if (p.second > hi) hi = p.second; }
            else { busy += (double)(hi - lo) * 1e-6; lo = p.first; hi = p.second; }
        }
        if (hi) busy += (double)(hi - lo) * 1e-6;
        Acc b; b.name = "stamped_busy"; b.n = iv.size(); b.ms = busy; acc.push_back(b);
        if (!iv.empty()) {
            unsigned long long last = 0; for (auto &p : iv) if (p.second > last) last = p.second;
            Acc sp; sp.name = "stamped_span"; sp.n = 1; sp.ms = (double)(last - iv.front().first) * 1e-6; acc.push_back(sp);
        }
    }
    if (!ctx->prof.empty() && cudaEventSynchronize(ctx->prof.back().ev) != cudaSuccess)
        return fail(ctx, REVNET_E_CUDA, std::string("revnet_profile_summary: ") + cudaGetErrorString(cudaGetLastError()));
    for (size_t i = 1; i < ctx->prof.size(); i++) {
        const ProfRec &r = ctx->prof[i];
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ctx->prof[i - 1].ev, r.ev) != cudaSuccess) { cudaGetLastError(); continue; }
        std::string key = r.name;
        if (ctx->prof_detail) { char sfx[64]; snprintf(sfx, sizeof sfx, "|%.0f|%.0f", r.bytes, r.flops); key += sfx; }
        Acc *a = nullptr;
        for (auto &x : acc) if (x.name == key) { a = &x; break; }
        if (!a) { acc.push_back(Acc()); a = &acc.back(); a->name = key; }
        a->n++; a->ms += ms; a->bytes += r.bytes; a->flops += r.flops;
    }
    std::string out;
    char line[256];
    for (auto &a : acc) {
        snprintf(line, sizeof line, "%s\t%llu\t%.6f\t%.0f\t%.0f\n", a.name.c_str(), (unsigned long long)a.n, a.ms, a.bytes, a.flops);
        out += line;
    }
    if (needed) *needed = out.size() + 1;
    if (buflen) { size_t n = out.size() < buflen - 1 ? out.size() : buflen - 1; memcpy(buf, out.data(), n); buf[n] = 0; }
    return REVNET_OK;
}
