// Residual-function and reversible-block engine: sequences the kernels for
//   forward   y1 = x1 + F(x2); y2 = x2 + G(y1)                                   (Section 3.1)
//   backward  Algorithm 1: x2 = y2 - G(y1); backprop G; x1 = y1 - F(x2); backprop F
// The tensors a residual function produces while being recomputed stay in the workspace and
// feed its own backprop, so each conv layer costs four passes per step in all.
//
// Batch statistics.  A tensor-core convolution leaves the per-channel mean and 1/sqrt(var+eps) of
// what it stores (its epilogue sums them), so the BN that reads the tensor next needs no pass of
// its own.  Inside a function that always applies.  For the coupling state it applies when the
// caller hands Moments through (a stack does); otherwise the statistics of x2 and y1 are computed
// by the stand-alone reduction, in the forward and in the reversal alike, which keeps the
// recomputed F and G bit-identical to the forward ones.
#include "common.cuh"

// dispatch: tensor-core kernels take the shapes they support in mode 0, the fp32 kernels the rest
bool conv_fprop_tc(Exec &ex, const void *a, Geom gi, const Layer &L, Pair out, Pair partner, int sign, Moments *stats);
bool conv_dgrad_tc(Exec &ex, const void *g, Geom gi, const Layer &L, float *da, const BnBwdReq *bb);
bool conv_dgrad_tc_s2(Exec &ex, const void *g, Geom gi, const Layer &L, float *da, const BnBwdReq *bb, bool *fused);
bool conv_wgrad_tc(Exec &ex, const void *g, const void *a, Geom gi, const Layer &L, float *dW, float *scratch, size_t *need);
bool conv_wgrad_tc_batch(Exec &ex, int n, const void *const *gq, const void *const *a, const Geom *gi, const Layer *const *L,
                         float *scratch, size_t *need);
// one kernel for BN -> ReLU -> conv (at most 64 input channels, stride 1); likewise the data gradient of such a layer
bool conv_fprop_fused(Exec &ex, Pair t, BnRef bn, Geom gi, const Layer &L, Pair out, Pair partner, int sign, Moments *stats, bf16 *a_out);
bool conv_dgrad_fused(Exec &ex, const void *g, Geom gi, const Layer &L, float *da, const BnBwdReq *bb);

// stats: in = where the statistics of `out` should go (or nullptr); stats->valid says whether the kernel provides them
static void conv_fprop(Exec &ex, const void *a, Geom gi, const Layer &L, Pair out, Pair partner, int sign, Moments *stats) {
    const bool b16 = ex.mode == 0;
    if (stats) stats->valid = false;
    if (b16 && conv_fprop_tc(ex, a, gi, L, out, partner, sign, stats)) return;
    if (stats) stats->valid = false;
    conv_fprop_simt(ex, a, b16, gi, L, out, partner, sign);
}
// returns true when the epilogue also produced the BN-backward sums asked for in bb
static bool conv_dgrad(Exec &ex, const void *g, Geom gi, const Layer &L, float *da, const BnBwdReq *bb) {
    const bool b16 = ex.mode == 0;
    if (b16 && L.stride == 1 && conv_dgrad_fused(ex, g, gi, L, da, bb)) return bb != nullptr;
    if (b16 && L.stride == 1 && conv_dgrad_tc(ex, g, gi, L, da, bb)) return bb != nullptr;
    // stride 2 on the tensor cores: the CTAs of one launch split into the parity classes of the input pixels
    bool fused = false;
    if (b16 && L.stride == 2 && L.cout % 8 == 0 && conv_dgrad_tc_s2(ex, g, gi, L, da, bb, &fused)) return fused;
    if (b16 && L.stride == 2 && gi.H % 2 == 0 && gi.W % 2 == 0 && L.cout % 8 == 0) {
        // shapes the class launches do not take: spread g over the input grid (zeros between samples); the data gradient is then the
        // stride-1 one:  da[y,x] = sum_taps g_up[y + pad - kh, x + pad - kw] W[.,kh,kw,.]
        size_t m = ex.ws.mark();
        bf16 *gup = ex.ws.get<bf16>(gi.P() * L.cout);
        upsample_zero_bf16(ex, (const bf16 *)g, gup, gi.N, gi.H / 2, gi.W / 2, L.cout);
        Layer L1 = L; L1.stride = 1;
        const bool ok = conv_dgrad_tc(ex, gup, gi, L1, da, bb);
        ex.ws.release(m);
        if (ok) return bb != nullptr;
    }
    conv_dgrad_simt(ex, g, b16, gi, L, da);
    return false;
}
static void conv_wgrad(Exec &ex, const void *g, const void *a, Geom gi, const Layer &L, float *dW) {
    const bool b16 = ex.mode == 0;
    if (b16 && conv_wgrad_tc(ex, g, a, gi, L, dW, nullptr, nullptr)) return;
    conv_wgrad_simt(ex, g, b16, a, b16, gi, L, dW);
}

static size_t esz(const Exec &ex) { return ex.mode == 0 ? 2 : 4; }

// out = partner + sign * Fn(u).  With `saved`, every layer's activated input, BN input and BN
// statistics are left in the workspace (the caller releases them after the backward).
void fn_forward(Exec &ex, Geom g, Pair u, const Moments *mom_in, const std::vector<Layer> &layers, Pair partner, Pair out,
                int sign, Moments *mom_out, FnSaved *saved, bool skip_last_conv) {
    const int L = (int)layers.size();
    const bool b16 = ex.mode == 0;
    size_t outer = ex.ws.mark();
    Pair t = u;
    Geom gi = g;
    if (saved) { saved->a.clear(); saved->t.clear(); saved->bn.clear(); saved->gin = g; }
    Moments cur;
    if (mom_in && mom_in->valid) cur = *mom_in;
    if (mom_out) mom_out->valid = false;
    for (int l = 0; l < L; l++) {
        const Layer &ly = layers[l];
        const size_t P = gi.P();
        if (!cur.valid) {
            cur = mom_alloc(ex, ly.cin);
            bn_stats(ex, t, P, cur);
            cur.valid = true;
        }
        const BnRef bn = bn_ref(ly.gamma, ly.beta, cur, ex.eps);
        const bool last = l == L - 1;
        Geom go{gi.N, conv_out(gi.H, ly.k, ly.stride), conv_out(gi.W, ly.k, ly.stride)};
        // the activated tensor is materialised only where something reads it: the unfused convolution, or the weight gradient
        void *a = ex.ws.alloc(P * ly.cin * esz(ex));
        float *tn = last ? nullptr : ex.ws.get<float>(go.P() * ly.cout);
        Moments next;
        if (!last) next = mom_alloc(ex, ly.cout, b16);      // with room for pending partials: the next layer consumes them
        const Pair o = last ? out : single(tn, ly.cout);
        bool fused = false;
        if (b16 && !(last && skip_last_conv))
            fused = conv_fprop_fused(ex, t, bn, gi, ly, o, last ? partner : Pair{}, last ? sign : 0, last ? mom_out : &next,
                                     saved ? (bf16 *)a : nullptr);
        if (fused) cur.pending = false;     // the fused kernel has stored mean and rstd
        else { mom_finalize(ex, cur, ly.cin); bn_relu_apply(ex, t, P, BnRef{ly.gamma, ly.beta, cur.mean, cur.rstd}, a, b16); }
        if (saved) { saved->a.push_back(a); saved->bn.push_back(cur); }
        if (last) {
            if (!skip_last_conv && !fused) conv_fprop(ex, a, gi, ly, out, partner, sign, mom_out);
        } else {
            if (!fused) conv_fprop(ex, a, gi, ly, single(tn, ly.cout), Pair{}, 0, &next);
            if (saved) saved->t.push_back(tn);
            t = single(tn, ly.cout);
            cur = next;     // valid only if the epilogue summed them; else the next round computes them
        }
        gi = go;
    }
    if (!saved) ex.ws.release(outer);
}

// dgin_out = add + (dFn/du)^T gup ; parameter gradients through the layers' pointers.
void fn_backward(Exec &ex, Geom g, Pair u, const std::vector<Layer> &layers, FnSaved &saved, Pair gup, const bf16 *gup_cast,
                 Pair add, Pair dgin_out, bf16 *dgin_cast) {
    const int L = (int)layers.size();
    const bool b16 = ex.mode == 0;
    size_t outer = ex.ws.mark();
    // geometry of every layer's input
    std::vector<Geom> gin(L + 1);
    gin[0] = g;
    for (int l = 0; l < L; l++)
        gin[l + 1] = Geom{gin[l].N, conv_out(gin[l].H, layers[l].k, layers[l].stride), conv_out(gin[l].W, layers[l].k, layers[l].stride)};
    // upstream gradient as one operand tensor
    const void *gcur;
    {
        const int C = gup.C();
        if (b16 && gup_cast) gcur = gup_cast;
        else if (!b16 && gup.c1 == 0) gcur = gup.p0;
        else {
            void *buf = ex.ws.alloc(gin[L].P() * C * esz(ex));
            concat_cast(ex, gup, gin[L].P(), buf, b16);
            gcur = buf;
        }
    }
    // The weight gradients of the function's layers run as ONE launch on a side stream, beside the
    // last layer's data gradient: by then every operand exists (the gradient entering layer 0 is the
    // last one produced).  One launch amortises set-up and split partials over the layers; the split
    // partials get a buffer of their own for that time.  Functions of more than four layers, shapes
    // the tensor-core kernel does not take, and profiling runs go layer by layer on the main stream.
    bool side = b16 && ex.use_side && L <= 4 && (ex.dry || (ex.ctx->side_stream && !ex.ctx->profiling));
    size_t wg_need = 0;
    std::vector<const Layer *> lptr(L);
    std::vector<const void *> gq(L), aq(L);
    for (int l = 0; l < L; l++) { lptr[l] = &layers[l]; aq[l] = saved.a[l]; }
    if (side && !conv_wgrad_tc_batch(ex, L, gq.data(), aq.data(), gin.data(), lptr.data(), nullptr, &wg_need)) side = false;
    float *wg_scratch = side && wg_need ? ex.ws.get<float>(wg_need) : nullptr;
    for (int l = L - 1; l >= 0; l--) {
        const Layer &ly = layers[l];
        const size_t P = gin[l].P();
        gq[l] = gcur;
        if (!side) {
            conv_wgrad(ex, gcur, saved.a[l], gin[l], ly, ly.dW);
        } else if (l == 0) {
            cudaStream_t main = ex.stream;
            if (!ex.dry) {
                cudaEventRecord(ex.ctx->ev_fork, main);
                cudaStreamWaitEvent(ex.ctx->side_stream, ex.ctx->ev_fork, 0);
                ex.stream = ex.ctx->side_stream;
            }
            conv_wgrad_tc_batch(ex, L, gq.data(), aq.data(), gin.data(), lptr.data(), wg_scratch, nullptr);
            ex.stream = main;
        }
        float *da = ex.ws.get<float>(P * ly.cin);
        float *coef = ex.ws.get<float>((size_t)3 * ly.cin);
        const Pair tl = l == 0 ? u : single(saved.t[l - 1], ly.cin);
        const BnRef bn{ly.gamma, ly.beta, saved.bn[l].mean, saved.bn[l].rstd};
        const BnBwdReq bb{tl, bn, ly.dgamma, ly.dbeta, coef};
        const bool sums_done = conv_dgrad(ex, gcur, gin[l], ly, da, &bb);
        if (l == 0) {
            // add.p0 == nullptr: the gradient is stored without a partner (stored transitions)
            bn_relu_bwd(ex, da, tl, P, bn, ly.dgamma, ly.dbeta, coef, sums_done, nullptr, false, add, dgin_out, b16 ? dgin_cast : nullptr);
        } else {
            void *dt = ex.ws.alloc(P * ly.cin * esz(ex));
            bn_relu_bwd(ex, da, tl, P, bn, ly.dgamma, ly.dbeta, coef, sums_done, dt, b16, Pair{}, Pair{}, nullptr);
            gcur = dt;
        }
    }
    if (side && !ex.dry) {
        cudaEventRecord(ex.ctx->ev_join, ex.ctx->side_stream);
        cudaStreamWaitEvent(ex.stream, ex.ctx->ev_join, 0);
    }
    ex.ws.release(outer);
}

void block_forward(Exec &ex, Geom g, int c, const std::vector<Layer> &F, const std::vector<Layer> &G,
                   float *x1, float *x2, float *y1, float *y2, const Moments *mx2, Moments *my1, Moments *my2) {
    const float q = ex.q;
    // without hand-off (stand-alone call) the statistics of x2 and y1 come from the stand-alone reduction,
    // as they will in the reversal, which is handed y1 from outside
    fn_forward(ex, g, single(x2, c, q), mx2, F, single(x1, c, q), single(y1, c, q), +1, my1, nullptr, false);
    fn_forward(ex, g, single(y1, c, q), my1, G, single(x2, c, q), single(y2, c, q), +1, my2, nullptr, false);
}

void block_backward(Exec &ex, Geom g, int c, const std::vector<Layer> &F, const std::vector<Layer> &G,
                    const float *y1, const float *y2, const float *dy1, const float *dy2,
                    float *x1, float *x2, float *dx1, float *dx2,
                    Moments *m1, Moments *m2, const Moments *m2_use, const bf16 *dy2_cast, bf16 *dx2_cast,
                    Moments *m1_out, bool overlap) {
    FnSaved svG, svF;
    const float q = ex.q;   // format of the coupling state; gradients are always float
    size_t m0 = ex.ws.mark();
    if (!m1_out) m1_out = m1;
    // F may be recomputed beside G's gradient steps only if it leaves y1 and its statistics alone
    overlap = overlap && x1 != y1 && m1_out != m1 && (ex.dry || (ex.ctx->recon_stream && !ex.ctx->profiling));
    // bf16 copy of dz1 for F's backward (the BN-backward apply that produces dz1 writes it)
    bf16 *dz1_cast = ex.mode == 0 ? ex.ws.get<bf16>(g.P() * c) : nullptr;
    size_t m = ex.ws.mark();
    // x2 = y2 - G(z1), z1 = y1
    fn_forward(ex, g, single((float *)y1, c, q), m1, G, single((float *)y2, c, q), single(x2, c, q), -1, m2, &svG, false);
    const Moments *mf = (m2_use && m2_use->valid) ? m2_use : m2;
    if (!overlap) {
        // dz1 = dy1 + (dG/dz1)^T dy2 ; dW_G
        fn_backward(ex, g, single((float *)y1, c, q), G, svG, single((float *)dy2, c), dy2_cast, single((float *)dy1, c), single(dx1, c), dz1_cast);
        ex.ws.release(m);
        // x1 = z1 - F(x2)
        fn_forward(ex, g, single(x2, c, q), mf, F, single((float *)y1, c, q), single(x1, c, q), -1, m1_out, &svF, false);
    } else {
        // x1 = z1 - F(x2) on the reconstruction stream (it needs x2 only), dz1 and dW_G meanwhile on the main stream;
        // F's internals are placed before G's gradient steps take their temporaries, so the arena stays a stack
        cudaStream_t main = ex.stream;
        if (!ex.dry) {
            cudaEventRecord(ex.ctx->ev_rfork, main);
            cudaStreamWaitEvent(ex.ctx->recon_stream, ex.ctx->ev_rfork, 0);
            ex.stream = ex.ctx->recon_stream;
        }
        // launches take short-lived scratch from the arena and hand it back at once, which is safe within one stream
        // only: what F's recomputation touched stays out of reach of the main stream's launches until the join
        ex.ws.high = ex.ws.off;
        fn_forward(ex, g, single(x2, c, q), mf, F, single((float *)y1, c, q), single(x1, c, q), -1, m1_out, &svF, false);
        if (ex.ws.high > ex.ws.off) ex.ws.off = ex.ws.high;
        if (!ex.dry) { cudaEventRecord(ex.ctx->ev_rjoin, ex.ctx->recon_stream); ex.stream = main; }
        fn_backward(ex, g, single((float *)y1, c, q), G, svG, single((float *)dy2, c), dy2_cast, single((float *)dy1, c), single(dx1, c), dz1_cast);
        if (!ex.dry) cudaStreamWaitEvent(main, ex.ctx->ev_rjoin, 0);
    }
    // dx2 = dy2 + (dF/dx2)^T dz1 ; dW_F ; dx1 = dz1 (already in place)
    fn_backward(ex, g, single(x2, c, q), F, svF, single(dx1, c), dz1_cast, single((float *)dy2, c), single(dx2, c), dx2_cast);
    ex.ws.release(m0);
}
