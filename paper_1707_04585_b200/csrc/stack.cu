// Stack driver: a classification network of reversible stages that keeps only the inputs of its
// non-reversible layers (Section 3.2).  Each stage owns ONE (x1,x2) buffer pair; its units run in
// place on it in the forward pass, and Algorithm 1 walks it back in place in the backward pass,
// so the activation footprint does not depend on the number of units.
#include "common.cuh"
#include <utility>
#include <string.h>
#include <array>
#include <stdlib.h>
#include <math.h>

struct LayerSlot {
    int cin, cout, k, stride; size_t off_gamma, off_beta, off_W;   // offsets in floats; stem: gamma/beta unused
    const bf16 *wp_f = nullptr, *wp_d = nullptr;                  // bf16 packs of the current step (mode 0)
};

struct StagePlan {
    int c, H, units;
    bool has_trans;
    LayerSlot trans;
    bool has_down = false;          // the stage starts with a stored down-sampling unit (paper-shaped stage)
    std::vector<LayerSlot> dF, dG;
    std::vector<std::vector<LayerSlot>> F, G;
    size_t off_x1, off_x2;          // bytes into the activation buffer
    size_t off_v1, off_v2;          // verify copies (bytes), valid with verify_reconstruction
};

struct revnet_plan {
    revnet_ctx *ctx;
    revnet_stack_desc d;
    LayerSlot stem;
    int stemH;                      // stem output resolution
    int poolH;                      // after max-pool (== stemH without)
    bool stem_direct;               // stem writes straight into stage 0's pair
    size_t off_stem_out, off_pool_out;
    std::vector<StagePlan> st;
    size_t off_fcW, off_fcb;
    int feat_C;
    size_t n_params, act_bytes, ws_bytes, param_scratch_bytes = 0;
    uint64_t stored_bytes;
    std::vector<uint32_t> seg_end; std::vector<uint8_t> seg_decay;
    void *pinned = nullptr;         // seg_end then seg_decay, page-locked for async upload
    bool pinned_is_malloc = false;  // no CUDA device at plan time: plain host memory instead
    void *pack_host = nullptr;      // page-locked staging for the weight-pack job table
    size_t pack_host_bytes = 0;
    // the step captured as a CUDA graph, valid for one set of buffer addresses
    size_t bound_act = 0, bound_ws = 0;   // sizes of the caller's buffers, if declared (revnet_plan_set_buffer_sizes)
    bool bound = false;
    cudaGraphExec_t graph_exec = nullptr;
    const void *graph_key[10] = {};
    bool graph_stamping = false;    // the captured step carries timeline stamps
    revnet_step_stats graph_stats = {};
};

static std::vector<std::array<int, 3>> fn_shape(int kind, int c, int w) {
    if (kind == 0) return {{c, c, 3}};
    if (kind == 1) return {{c, c, 3}, {c, c, 3}};
    return {{c, w, 1}, {w, w, 3}, {w, c, 1}};
}

static Layer bind(const LayerSlot &s, float *params, float *grads) {
    Layer L;
    L.cin = s.cin; L.cout = s.cout; L.k = s.k; L.stride = s.stride;
    L.W = params + s.off_W; L.gamma = params + s.off_gamma; L.beta = params + s.off_beta;
    L.dW = grads + s.off_W; L.dgamma = grads + s.off_gamma; L.dbeta = grads + s.off_beta;
    L.Wp_fprop = s.wp_f; L.Wp_dgrad = s.wp_d;
    return L;
}
static std::vector<Layer> bind(const std::vector<LayerSlot> &v, float *params, float *grads) {
    std::vector<Layer> o;
    for (auto &s : v) o.push_back(bind(s, params, grads));
    return o;
}

// Runs (or, with ex.dry, only sizes) one training step.
static void run_step(revnet_plan *pl, Exec &ex, const float *images, const int32_t *labels, float *params, float *grads,
                     float *mom, char *act, float *loss, int32_t *pred, float *logits_out, revnet_step_stats *stats,
                     float **recon_dev) {
    const revnet_stack_desc &d = pl->d;
    const int N = d.N, S = d.n_stages;
    auto actf = [&](size_t off) { return (float *)(act + off); };
    const float q = ex.q;   // format of the stage buffers (the coupling state)

    ex.mark("step_begin");
    if (!ex.dry && ex.ctx->stamping && ex.ctx->stamps) {
        // a step's stamps start from "no start yet" (all ones) and "no end yet" (zero); part of the captured graph
        cudaMemsetAsync(ex.ctx->stamps, 0xff, kStampSlots * sizeof(unsigned long long), ex.stream);
        cudaMemsetAsync(ex.ctx->stamps + kStampSlots, 0, kStampSlots * sizeof(unsigned long long), ex.stream);
        ex.ctx->stamp_next = 0;
        ex.ctx->stamp_recs.clear();
    }
    // ---- step-long scratch
    const size_t nseg = pl->seg_end.size();
    uint32_t *seg_end = ex.ws.get<uint32_t>(nseg);
    uint8_t *seg_decay = ex.ws.get<uint8_t>(nseg);
    if (!ex.dry) {
        cudaMemcpyAsync(seg_end, pl->pinned, nseg * 4, cudaMemcpyHostToDevice, ex.stream);
        cudaMemcpyAsync(seg_decay, (char *)pl->pinned + nseg * 4, nseg, cudaMemcpyHostToDevice, ex.stream);
    }
    // bf16 weight packs for the tensor-core kernels: every stride-1 BN-ReLU-conv layer, one launch
    {
        std::vector<LayerSlot *> slots;
        for (auto &s : pl->st) {
            if (s.has_trans) slots.push_back(&s.trans);
            for (auto &l : s.dF) slots.push_back(&l);
            for (auto &l : s.dG) slots.push_back(&l);
            for (auto &f : s.F) for (auto &l : f) slots.push_back(&l);
            for (auto &f : s.G) for (auto &l : f) slots.push_back(&l);
        }
        std::vector<PackJob> jobs;
        double bytes = 0;
        size_t max_elems = 0;
        for (LayerSlot *l : slots) {
            l->wp_f = l->wp_d = nullptr;
            if (ex.mode != 0 || l->cin % 8 || l->cout % 8) continue;
            size_t nf = tc_pack_elems(l->cin, l->cout, l->k, false), nd = tc_pack_elems(l->cin, l->cout, l->k, true);
            bf16 *f = ex.ws.get<bf16>(nf), *dd = ex.ws.get<bf16>(nd);
            l->wp_f = f; l->wp_d = dd;
            jobs.push_back(tc_pack_job(params + l->off_W, f, l->cin, l->cout, l->k, false));
            jobs.push_back(tc_pack_job(params + l->off_W, dd, l->cin, l->cout, l->k, true));
            bytes += (double)(nf + nd) * 2 + (double)l->cin * l->cout * l->k * l->k * 8;
            if (nf > max_elems) max_elems = nf;
            if (nd > max_elems) max_elems = nd;
        }
        PackJob *jobs_dev = ex.ws.get<PackJob>(jobs.size() + 1);
        if (!ex.dry && !jobs.empty()) {
            if (jobs.size() * sizeof(PackJob) <= pl->pack_host_bytes) {
                memcpy(pl->pack_host, jobs.data(), jobs.size() * sizeof(PackJob));
                cudaMemcpyAsync(jobs_dev, pl->pack_host, jobs.size() * sizeof(PackJob), cudaMemcpyHostToDevice, ex.stream);
                tc_pack_batch(ex, jobs_dev, (int)jobs.size(), bytes, max_elems);
            } else {
                for (LayerSlot *l : slots) l->wp_f = l->wp_d = nullptr;   // no staging room: pack per call instead
            }
        }
    }
    if (ex.dry) pl->param_scratch_bytes = (ex.ws.off + 255) & ~size_t(255);   // everything above scales with the parameters, not the activations
    size_t gmax = (size_t)N * pl->stemH * pl->stemH * d.stem_cout;           // gradient w.r.t. stem / pool output
    for (auto &s : pl->st) { size_t e = (size_t)N * s.H * s.H * 2 * s.c; if (e > gmax) gmax = e; }
    float *gbuf[2] = {ex.ws.get<float>(gmax), ex.ws.get<float>(gmax)};
    const int K = d.n_classes, FC = pl->feat_C;
    float *feat = ex.ws.get<float>((size_t)N * FC), *dfeat = ex.ws.get<float>((size_t)N * FC);
    float *logits = logits_out ? logits_out : ex.ws.get<float>((size_t)N * K);
    float *dlogits = ex.ws.get<float>((size_t)N * K);
    // batch statistics handed from kernel to kernel: per stage those of the current (x1,x2) pair (one
    // [2c] array each for mean and rstd, so that the pair reads as one tensor to a transition) and
    // those of the stage's input x2, which the reversal of the first unit needs again
    struct StageMom { Moments m1, m2, cat, in_cat, in2, dy1; };      // dy1: statistics of a down-sampling unit's y1, kept for its backward
    std::vector<StageMom> sm(S);
    bf16 *gcast = nullptr;          // bf16 copy of the gradient w.r.t. x2 / y2, handed from unit to unit
    float *x1_alt = nullptr, *m1_alt_buf = nullptr;
    bf16 *gcast2 = nullptr;         // stored-activation step: bf16 copy of the gradient w.r.t. z1 inside a unit
    // Stored-activation step (ordinary backprop): what every unit keeps from the forward pass.  The tensors
    // live in the workspace arena, unit after unit, and are released in reverse order by the backward pass.
    struct StoredUnit { size_t mark; float *x1, *x2, *y1, *y2; FnSaved svF, svG; Moments my1, my2; };
    std::vector<std::vector<StoredUnit>> kept(S);
    std::vector<Pair> stage_out(S);
    const bool stored = d.store_activations != 0;
    uint64_t kept_bytes = 0;        // what the units keep, summed over the network
    {
        size_t cmax = 0;
        for (int si = 0; si < S; si++) {
            const StagePlan &s = pl->st[si];
            float *b = ex.ws.get<float>((size_t)10 * s.c);
            sm[si].dy1.mean = b + 8 * s.c; sm[si].dy1.rstd = b + 9 * s.c;
            sm[si].cat.mean = b; sm[si].cat.rstd = b + 2 * s.c;
            sm[si].m1.mean = b; sm[si].m1.rstd = b + 2 * s.c;
            sm[si].m2.mean = b + s.c; sm[si].m2.rstd = b + 3 * s.c;
            sm[si].in_cat.mean = b + 4 * s.c; sm[si].in_cat.rstd = b + 6 * s.c;
            sm[si].in2.mean = b + 5 * s.c; sm[si].in2.rstd = b + 7 * s.c;
            size_t e = (size_t)N * s.H * s.H * s.c; if (e > cmax) cmax = e;
        }
        if (ex.mode == 0) gcast = ex.ws.get<bf16>(cmax);
        // the reversal writes x1 beside y1 instead of over it (the two buffers change roles from unit to unit), and the
        // statistics of x1 beside those of y1, so that F can be recomputed while G's gradient steps still read y1
        if (!d.store_activations) { x1_alt = ex.ws.get<float>(cmax); size_t c2 = 0; for (auto &st : pl->st) if ((size_t)st.c > c2) c2 = st.c; m1_alt_buf = ex.ws.get<float>(2 * c2); }
        if (ex.mode == 0 && d.store_activations) gcast2 = ex.ws.get<bf16>(cmax);
    }
    float *recon = ex.ws.get<float>(REVNET_MAX_STAGES);
    if (recon_dev) *recon_dev = recon;
    if (d.verify_reconstruction) fill_zero(ex, recon, REVNET_MAX_STAGES * sizeof(float));

    // ---- forward
    Layer stem = bind(pl->stem, params, grads);
    Geom gimg{N, d.img, d.img};
    StagePlan &s0 = pl->st[0];
    {
        const Pair so = pl->stem_direct ? halves(actf(s0.off_x1), actf(s0.off_x2), s0.c, q) : single(actf(pl->off_stem_out), d.stem_cout);
        if (!stem_fprop(ex, images, gimg, stem, so)) conv_fprop_simt(ex, images, false, gimg, stem, so, Pair{}, 0);
    }
    Pair prev = single(actf(pl->off_stem_out), d.stem_cout);
    int prevH = pl->stemH;
    if (d.maxpool) {
        maxpool_fwd(ex, actf(pl->off_stem_out), actf(pl->off_pool_out), N, pl->stemH, pl->stemH, d.stem_cout);
        prev = single(actf(pl->off_pool_out), d.stem_cout);
        prevH = pl->poolH;
    }
    for (int si = 0; si < S; si++) {
        StagePlan &s = pl->st[si];
        float *x1 = actf(s.off_x1), *x2 = actf(s.off_x2);
        Geom g{N, s.H, s.H};
        StageMom &mo = sm[si];
        if (s.has_trans) {
            std::vector<Layer> T{bind(s.trans, params, grads)};
            const Moments *min = si > 0 ? &sm[si - 1].cat : nullptr;
            fn_forward(ex, Geom{N, prevH, prevH}, prev, min, T, Pair{}, halves(x1, x2, s.c, q), 0, &mo.in_cat, nullptr, false);
        }
        mo.in2.valid = mo.in_cat.valid;
        if (s.has_down) {
            // y1 = S(x1) + F(x2); y2 = S(x2) + G(y1) on the pair of the stage in front, which stays where it is (stored)
            StagePlan &pv = pl->st[si - 1];
            const Geom gp{N, pv.H, pv.H};
            size_t m = ex.ws.mark();
            float *sc = ex.ws.get<float>(g.P() * s.c);
            shortcut_fwd(ex, prev.p0, sc, N, pv.H, pv.H, pv.c, s.c, q);
            fn_forward(ex, gp, single(prev.p1, pv.c, q), &sm[si - 1].m2, bind(s.dF, params, grads), single(sc, s.c, q), single(x1, s.c, q), +1, &mo.dy1, nullptr, false);
            if (!mo.dy1.valid) { bn_stats(ex, single(x1, s.c, q), g.P(), mo.dy1); mo.dy1.valid = true; }
            shortcut_fwd(ex, prev.p1, sc, N, pv.H, pv.H, pv.c, s.c, q);
            fn_forward(ex, g, single(x1, s.c, q), &mo.dy1, bind(s.dG, params, grads), single(sc, s.c, q), single(x2, s.c, q), +1, &mo.in2, nullptr, false);
            ex.ws.release(m);
        }
        if (!mo.in2.valid) { bn_stats(ex, single(x2, s.c, q), g.P(), mo.in2); mo.in2.valid = true; }
        if (d.verify_reconstruction && !ex.dry) {
            size_t b = g.P() * s.c * sizeof(float);
            cudaMemcpyAsync(actf(s.off_v1), x1, b, cudaMemcpyDeviceToDevice, ex.stream);
            cudaMemcpyAsync(actf(s.off_v2), x2, b, cudaMemcpyDeviceToDevice, ex.stream);
        }
        if (!stored) {
            for (int u = 0; u < s.units; u++)
                block_forward(ex, g, s.c, bind(s.F[u], params, grads), bind(s.G[u], params, grads), x1, x2, x1, x2,
                              u == 0 ? &mo.in2 : &mo.m2, &mo.m1, &mo.m2);
            mo.cat.valid = mo.m1.valid && mo.m2.valid;
            prev = halves(x1, x2, s.c, q);
        } else {
            // every unit writes its outputs to fresh tensors and leaves the internals of F and G where they are
            kept[si].resize(s.units);
            float *c1 = x1, *c2 = x2;
            const Moments *m_in = &mo.in2;
            const size_t half = g.P() * s.c;
            for (int u = 0; u < s.units; u++) {
                StoredUnit &k = kept[si][u];
                k.mark = ex.ws.mark();
                k.x1 = c1; k.x2 = c2;
                const bool last_unit = u == s.units - 1;
                k.y1 = ex.ws.get<float>(half); k.y2 = ex.ws.get<float>(half);
                // the statistics of the stage's final pair go where the next transition expects them
                if (last_unit) { k.my1 = mo.m1; k.my2 = mo.m2; }
                else { k.my1 = mom_alloc(ex, s.c); k.my2 = mom_alloc(ex, s.c); }
                fn_forward(ex, g, single(c2, s.c, q), m_in, bind(s.F[u], params, grads), single(c1, s.c, q), single(k.y1, s.c, q), +1, &k.my1, &k.svF, false);
                fn_forward(ex, g, single(k.y1, s.c, q), &k.my1, bind(s.G[u], params, grads), single(c2, s.c, q), single(k.y2, s.c, q), +1, &k.my2, &k.svG, false);
                if (last_unit) { mo.m1 = k.my1; mo.m2 = k.my2; }
                c1 = k.y1; c2 = k.y2; m_in = &k.my2;
                kept_bytes += ex.ws.mark() - k.mark;
            }
            mo.cat.valid = mo.m1.valid && mo.m2.valid;
            prev = halves(c1, c2, s.c, q);
        }
        stage_out[si] = prev;
        prevH = s.H;
    }
    StagePlan &top = pl->st[S - 1];
    head_fwd(ex, prev, N, top.H * top.H, params + pl->off_fcW, params + pl->off_fcb, labels, K, feat, logits, dlogits, loss, pred);
    const uint64_t flops_fwd = ex.flops;

    // ---- backward
    int gi = (S - 1) & 1;
    {
        size_t half = (size_t)N * top.H * top.H * top.c;
        head_bwd(ex, halves(gbuf[gi], gbuf[gi] + half, top.c), N, top.H * top.H, params + pl->off_fcW, feat, dlogits, K,
                 grads + pl->off_fcW, grads + pl->off_fcb, dfeat);
    }
    for (int si = S - 1; si >= 0; si--) {
        StagePlan &s = pl->st[si];
        float *x1 = actf(s.off_x1), *x2 = actf(s.off_x2);
        Geom g{N, s.H, s.H};
        size_t half = g.P() * s.c;
        float *d1 = gbuf[gi], *d2 = gbuf[gi] + half;
        StageMom &mo = sm[si];
        if (!stored) {
            Moments mcur = mo.m1, malt = mo.m1;
            malt.mean = m1_alt_buf; malt.rstd = m1_alt_buf + s.c; malt.valid = false;
            float *cur1 = x1, *alt1 = x1_alt;
            for (int u = s.units - 1; u >= 0; u--) {
                // x1 alternates between the two buffers from unit to unit
                block_backward(ex, g, s.c, bind(s.F[u], params, grads), bind(s.G[u], params, grads), cur1, x2, d1, d2, alt1, x2, d1, d2,
                               &mcur, &mo.m2, u == 0 ? &mo.in2 : nullptr, u == s.units - 1 ? nullptr : gcast, gcast, &malt, true);
                std::swap(cur1, alt1);
                std::swap(mcur, malt);
            }
            // after an odd number of units the stage's input sits in the other buffer: bring it home
            if (cur1 != x1 && !ex.dry) cudaMemcpyAsync(x1, cur1, g.P() * s.c * sizeof(float), cudaMemcpyDeviceToDevice, ex.stream);
        } else {
            // Algorithm 1 without its reconstruction lines: the gradient steps read what the forward pass kept
            for (int u = s.units - 1; u >= 0; u--) {
                StoredUnit &k = kept[si][u];
                fn_backward(ex, g, single(k.y1, s.c, q), bind(s.G[u], params, grads), k.svG, single(d2, s.c), u == s.units - 1 ? nullptr : gcast,
                            single(d1, s.c), single(d1, s.c), gcast2);
                fn_backward(ex, g, single(k.x2, s.c, q), bind(s.F[u], params, grads), k.svF, single(d1, s.c), gcast2,
                            single(d2, s.c), single(d2, s.c), gcast);
                ex.ws.release(k.mark);
            }
        }
        if (d.verify_reconstruction && !stored) {
            max_abs_diff(ex, x1, actf(s.off_v1), half, q, recon + si);
            max_abs_diff(ex, x2, actf(s.off_v2), half, q, recon + si);
        }
        if (s.has_down) {
            // ordinary backprop through the stored unit: G from y1 (what the reversal left in the stage's pair), F from the
            // kept pair of the stage in front; both with the statistics of the forward pass
            StagePlan &pv = pl->st[si - 1];
            const Geom gp{N, pv.H, pv.H};
            const Pair pin = stored ? stage_out[si - 1] : halves(actf(pv.off_x1), actf(pv.off_x2), pv.c, q);
            const size_t ph = gp.P() * pv.c;
            float *o1 = gbuf[gi ^ 1], *o2 = gbuf[gi ^ 1] + ph;
            size_t m = ex.ws.mark();
            bf16 *dz1_cast = ex.mode == 0 ? ex.ws.get<bf16>(g.P() * s.c) : nullptr;
            {
                FnSaved sv;
                size_t m2 = ex.ws.mark();
                std::vector<Layer> G = bind(s.dG, params, grads);
                fn_forward(ex, g, single(x1, s.c, q), &mo.dy1, G, Pair{}, Pair{}, 0, nullptr, &sv, true);
                // dz1 = dy1 + (dG/dy1)^T dy2, in place over d1
                fn_backward(ex, g, single(x1, s.c, q), G, sv, single(d2, s.c), nullptr, single(d1, s.c), single(d1, s.c), dz1_cast);
                ex.ws.release(m2);
            }
            shortcut_bwd(ex, d2, o2, N, pv.H, pv.H, pv.c, s.c);
            {
                FnSaved sv;
                size_t m2 = ex.ws.mark();
                std::vector<Layer> F = bind(s.dF, params, grads);
                fn_forward(ex, gp, single(pin.p1, pv.c, q), &sm[si - 1].m2, F, Pair{}, Pair{}, 0, nullptr, &sv, true);
                // dx2 = S^T dy2 + (dF/dx2)^T dz1
                fn_backward(ex, gp, single(pin.p1, pv.c, q), F, sv, single(d1, s.c), dz1_cast, single(o2, pv.c), single(o2, pv.c), nullptr);
                ex.ws.release(m2);
            }
            shortcut_bwd(ex, d1, o1, N, pv.H, pv.H, pv.c, s.c);     // dx1 = S^T dz1
            ex.ws.release(m);
            gi ^= 1;
        }
        if (s.has_trans) {
            std::vector<Layer> T{bind(s.trans, params, grads)};
            Pair tin; int tH; Pair gout;
            if (si > 0) {
                StagePlan &p = pl->st[si - 1];
                tin = stored ? stage_out[si - 1] : halves(actf(p.off_x1), actf(p.off_x2), p.c, q); tH = p.H;
                size_t ph = (size_t)N * p.H * p.H * p.c;
                gout = halves(gbuf[gi ^ 1], gbuf[gi ^ 1] + ph, p.c);
            } else {
                tin = single(actf(d.maxpool ? pl->off_pool_out : pl->off_stem_out), d.stem_cout); tH = pl->poolH;
                gout = single(gbuf[gi ^ 1], d.stem_cout);
            }
            FnSaved sv;
            size_t m = ex.ws.mark();
            // rebuild the operands from the stored input (the stage in front still holds its forward statistics)
            fn_forward(ex, Geom{N, tH, tH}, tin, si > 0 ? &sm[si - 1].cat : nullptr, T, Pair{}, Pair{}, 0, nullptr, &sv, true);
            fn_backward(ex, Geom{N, tH, tH}, tin, T, sv, halves(d1, d2, s.c), nullptr, Pair{}, gout, nullptr);
            ex.ws.release(m);
            gi ^= 1;
        }
    }
    // gradient w.r.t. the stem output now sits in gbuf[gi]: a pair if the stem feeds stage 0 directly
    {
        size_t m = ex.ws.mark();
        const float *gstem;
        size_t Pstem = (size_t)N * pl->stemH * pl->stemH;
        if (pl->stem_direct) {
            float *cat = ex.ws.get<float>(Pstem * d.stem_cout);
            concat_cast(ex, halves(gbuf[gi], gbuf[gi] + Pstem * s0.c, s0.c), Pstem, cat, false);
            gstem = cat;
        } else if (d.maxpool) {
            float *gp = ex.ws.get<float>(Pstem * d.stem_cout);
            maxpool_bwd(ex, actf(pl->off_stem_out), gbuf[gi], gp, N, pl->stemH, pl->stemH, d.stem_cout);
            gstem = gp;
        } else {
            gstem = gbuf[gi];
        }
        if (!stem_wgrad(ex, images, gstem, gimg, stem, stem.dW)) conv_wgrad_simt(ex, gstem, false, images, false, gimg, stem, stem.dW);
        ex.ws.release(m);
    }
    bool quads = true;
    for (size_t i = 0; i + 1 < nseg; i++) quads = quads && pl->seg_end[i] % 4 == 0;
    sgd_update(ex, params, grads, mom, pl->n_params, seg_end, seg_decay, (int)nseg, d.lr, d.momentum, d.weight_decay, quads);

    if (stats) {
        stats->stored_activation_bytes = pl->stored_bytes + kept_bytes;
        stats->workspace_peak_bytes = ex.ws.peak;
        stats->flops_fwd = flops_fwd;
        stats->flops_bwd = ex.flops - flops_fwd;
        stats->kernel_launches = ex.launches;
        stats->device_status = 0;
        for (int i = 0; i < REVNET_MAX_STAGES; i++) stats->recon_max_abs[i] = 0.f;
    }
}

static int fail(revnet_ctx *ctx, int code, const std::string &msg) { if (ctx) ctx->err = msg; return code; }

extern "C" int revnet_stack_plan(revnet_ctx *ctx, const revnet_stack_desc *desc, revnet_plan **plan_out,
                                 size_t *param_count, size_t *activation_bytes, size_t *workspace_bytes) {
    if (!ctx || !desc || !plan_out) return fail(ctx, REVNET_E_INVALID_ARG, "revnet_stack_plan: null argument");
    const revnet_stack_desc &d = *desc;
    if (d.N < 1 || d.img < 1 || d.in_ch < 1 || d.n_classes < 2 || d.n_stages < 1 || d.n_stages > REVNET_MAX_STAGES)
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_stack_plan: bad N/img/in_ch/n_classes/n_stages");
    if ((d.stem_k != 3 && d.stem_k != 7) || (d.stem_stride != 1 && d.stem_stride != 2) || d.stem_cout % 4)
        return fail(ctx, REVNET_E_UNSUPPORTED_SHAPE, "revnet_stack_plan: stem must be 3x3 or 7x7, stride 1 or 2, cout % 4 == 0");
    if (d.mode != 0 && d.mode != 1) return fail(ctx, REVNET_E_INVALID_ARG, "revnet_stack_plan: mode must be 0 or 1");
    if (d.state_frac_bits < 0 || d.state_frac_bits > 24) return fail(ctx, REVNET_E_INVALID_ARG, "revnet_stack_plan: state_frac_bits must be in [0,24]");
    revnet_plan *pl = new revnet_plan();
    pl->ctx = ctx; pl->d = d;
    size_t off = 0;
    auto take = [&](size_t n, bool decay) { size_t o = off; off += n; pl->seg_end.push_back((uint32_t)off); pl->seg_decay.push_back(decay); return o; };
    auto slot = [&](int cin, int cout, int k, int stride, bool bn) {
        LayerSlot s;
        s.cin = cin; s.cout = cout; s.k = k; s.stride = stride; s.off_gamma = s.off_beta = s.off_W = 0;
        if (bn) { s.off_gamma = take(cin, false); s.off_beta = take(cin, false); }
        s.off_W = take((size_t)cout * k * k * cin, true);
        return s;
    };
    pl->stem = slot(d.in_ch, d.stem_cout, d.stem_k, d.stem_stride, false);
    pl->stemH = conv_out(d.img, d.stem_k, d.stem_stride);
    pl->poolH = d.maxpool ? conv_out(pl->stemH, 3, 2) : pl->stemH;
    int cprev = d.stem_cout, H = pl->poolH;
    size_t aoff = 0;
    auto atake = [&](size_t bytes) { size_t o = aoff; aoff += (bytes + 255) & ~size_t(255); return o; };
    pl->stem_direct = !d.maxpool && d.stage[0].trans_k == 0;
    pl->stored_bytes = (uint64_t)d.N * d.img * d.img * d.in_ch * 4;
    pl->off_stem_out = pl->off_pool_out = 0;
    if (!pl->stem_direct) {
        size_t b = (size_t)d.N * pl->stemH * pl->stemH * d.stem_cout * 4;
        pl->off_stem_out = atake(b); pl->stored_bytes += b;
        if (d.maxpool) { size_t pb = (size_t)d.N * H * H * d.stem_cout * 4; pl->off_pool_out = atake(pb); pl->stored_bytes += pb; }
    }
    for (int si = 0; si < d.n_stages; si++) {
        const revnet_stage_desc &sd = d.stage[si];
        bool bad = sd.units < 1 || sd.c < 4 || sd.c % 4 || sd.kind < 0 || sd.kind > 2 || (sd.kind == 2 && (sd.w < 4 || sd.w % 4));
        bad = bad || (sd.trans_k != 0 && sd.trans_k != 1 && sd.trans_k != 3) || (sd.trans_k && sd.trans_stride != 1 && sd.trans_stride != 2);
        // a stage without a transition is only possible directly behind a stem that needs no pooling
        bad = bad || (sd.trans_k == 0 && !sd.down && (si > 0 || d.maxpool || cprev != 2 * sd.c));
        // a down-sampling first unit: not in stage 0, instead of a transition, on an even resolution, at least the width in front
        bad = bad || (sd.down && (si == 0 || sd.trans_k != 0 || sd.kind == 0 || H % 2 || 2 * sd.c < cprev || cprev % 8));
        if (bad) { delete pl; return fail(ctx, REVNET_E_UNSUPPORTED_SHAPE, "revnet_stack_plan: unsupported stage " + std::to_string(si)); }
        StagePlan s;
        s.c = sd.c; s.units = sd.units; s.has_trans = sd.trans_k != 0;
        if (s.has_trans) { s.trans = slot(cprev, 2 * sd.c, sd.trans_k, sd.trans_stride, true); H = conv_out(H, sd.trans_k, sd.trans_stride); }
        if (sd.down) {
            s.has_down = true;
            const int ch = cprev / 2;
            if (sd.kind == 1) { s.dF.push_back(slot(ch, sd.c, 3, 2, true)); s.dF.push_back(slot(sd.c, sd.c, 3, 1, true)); }
            else { s.dF.push_back(slot(ch, sd.w, 1, 1, true)); s.dF.push_back(slot(sd.w, sd.w, 3, 2, true)); s.dF.push_back(slot(sd.w, sd.c, 1, 1, true)); }
            for (auto &sh : fn_shape(sd.kind, sd.c, sd.w)) s.dG.push_back(slot(sh[0], sh[1], sh[2], 1, true));
            H /= 2;
        }
        s.H = H;
        s.units = sd.units - (sd.down ? 1 : 0);       // reversible units
        for (int u = 0; u < s.units; u++) {
            for (int f = 0; f < 2; f++) {
                std::vector<LayerSlot> v;
                for (auto &sh : fn_shape(sd.kind, sd.c, sd.w)) v.push_back(slot(sh[0], sh[1], sh[2], 1, true));
                (f == 0 ? s.F : s.G).push_back(v);
            }
        }
        size_t hb = (size_t)d.N * H * H * sd.c * 4;
        s.off_x1 = atake(hb); s.off_x2 = atake(hb);
        pl->stored_bytes += 2 * hb;
        s.off_v1 = s.off_v2 = 0;
        pl->st.push_back(s);
        cprev = 2 * sd.c;
    }
    if (d.verify_reconstruction)
        for (auto &s : pl->st) { size_t hb = (size_t)d.N * s.H * s.H * s.c * 4; s.off_v1 = atake(hb); s.off_v2 = atake(hb); }
    pl->feat_C = cprev;
    pl->off_fcW = take((size_t)d.n_classes * cprev, true);
    pl->off_fcb = take(d.n_classes, false);
    pl->n_params = off;
    pl->act_bytes = aoff;
    if (off >= 0xffffffffull) { delete pl; return fail(ctx, REVNET_E_UNSUPPORTED_SHAPE, "revnet_stack_plan: more than 2^32 parameters"); }
    size_t nseg = pl->seg_end.size();
    if (cudaMallocHost(&pl->pinned, nseg * 5) != cudaSuccess) {
        cudaGetLastError();
        pl->pinned = malloc(nseg * 5);
        pl->pinned_is_malloc = true;
        if (!pl->pinned) { delete pl; return fail(ctx, REVNET_E_INTERNAL, "revnet_stack_plan: out of host memory"); }
    }
    {
        size_t layers = 0;
        for (auto &st : pl->st) layers += 1 + 6 + (size_t)st.units * 6;
        pl->pack_host_bytes = layers * 2 * sizeof(PackJob);
        if (pl->pinned_is_malloc || cudaMallocHost(&pl->pack_host, pl->pack_host_bytes) != cudaSuccess) {
            cudaGetLastError(); pl->pack_host = nullptr; pl->pack_host_bytes = 0;
        }
    }
    memcpy(pl->pinned, pl->seg_end.data(), nseg * 4);
    memcpy((char *)pl->pinned + nseg * 4, pl->seg_decay.data(), nseg);
    // size the workspace with a dry run of the very same driver
    Exec ex; ex.ctx = ctx; ex.dry = true; ex.ws.dry = true; ex.mode = d.mode; ex.eps = d.eps;
    ex.q = d.state_frac_bits ? ldexpf(1.f, -d.state_frac_bits) : 0.f;
    run_step(pl, ex, nullptr, nullptr, (float *)0x1000, (float *)0x1000, (float *)0x1000, (char *)0x1000, nullptr, nullptr, nullptr, nullptr, nullptr);
    pl->ws_bytes = ex.ws.peak + 256;
    if (param_count) *param_count = pl->n_params;
    if (activation_bytes) *activation_bytes = pl->act_bytes;
    if (workspace_bytes) *workspace_bytes = pl->ws_bytes;
    *plan_out = pl;
    return REVNET_OK;
}

extern "C" int revnet_plan_scratch_split(const revnet_plan *pl, size_t *param_scratch_bytes, size_t *activation_scratch_bytes) {
    if (!pl) return REVNET_E_INVALID_ARG;
    if (param_scratch_bytes) *param_scratch_bytes = pl->param_scratch_bytes;
    if (activation_scratch_bytes) *activation_scratch_bytes = pl->ws_bytes - pl->param_scratch_bytes;
    return REVNET_OK;
}

extern "C" int revnet_plan_set_buffer_sizes(revnet_plan *pl, size_t activation_bytes, size_t workspace_bytes) {
    if (!pl) return REVNET_E_INVALID_ARG;
    pl->bound_act = activation_bytes; pl->bound_ws = workspace_bytes; pl->bound = true;
    return REVNET_OK;
}

// status word of the device as it stands (the caller has just synchronised the stream); not cleared here
static int read_device_status(revnet_ctx *ctx, cudaStream_t s) {
    int st = 0;
    if (!ctx->dev_status) return 0;
    if (cudaMemcpyAsync(&st, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return REVNET_E_CUDA;
    }
    return st;
}

extern "C" int revnet_plan_destroy(revnet_plan *pl) {
    if (!pl) return REVNET_OK;
    if (pl->pinned) { if (pl->pinned_is_malloc) free(pl->pinned); else cudaFreeHost(pl->pinned); }
    if (pl->graph_exec) cudaGraphExecDestroy(pl->graph_exec);
    if (pl->pack_host) cudaFreeHost(pl->pack_host);
    delete pl;
    return REVNET_OK;
}

extern "C" int revnet_train_step(revnet_ctx *ctx, revnet_plan *pl, const float *images, const int32_t *labels,
                                 float *params, float *grads, float *momentum, void *activations, void *workspace,
                                 float *loss, int32_t *pred, float *logits, revnet_step_stats *stats, void *stream) {
    if (!ctx || !pl || !images || !labels || !params || !grads || !momentum || !activations || !workspace || !loss || !pred)
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_train_step: null argument");
    const void *ptrs[] = {images, params, grads, momentum, activations, workspace};
    for (const void *p : ptrs)
        if ((uintptr_t)p & 15) return fail(ctx, REVNET_E_MISALIGNED, "revnet_train_step: pointers must be 16-byte aligned");
    if (pl->bound && (pl->bound_act < pl->act_bytes || pl->bound_ws < pl->ws_bytes))
        return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_train_step: buffers declared as " + std::to_string(pl->bound_act) + " / " +
                    std::to_string(pl->bound_ws) + " bytes (activations / workspace), the plan needs " + std::to_string(pl->act_bytes) + " / " + std::to_string(pl->ws_bytes));
    const bool use_graph = pl->d.use_cuda_graph && !pl->d.verify_reconstruction && !ctx->profiling && ctx->capture_stream;
    const void *key[10] = {images, labels, params, grads, momentum, activations, workspace, loss, pred, logits};
    if (use_graph && pl->graph_exec && memcmp(key, pl->graph_key, sizeof key) == 0 && pl->graph_stamping == ctx->stamping) {
        if (cudaGraphLaunch(pl->graph_exec, (cudaStream_t)stream) != cudaSuccess)
            return fail(ctx, REVNET_E_CUDA, std::string("revnet_train_step: graph launch: ") + cudaGetErrorString(cudaGetLastError()));
        if (stats) *stats = pl->graph_stats;
        return REVNET_OK;
    }
    Exec ex; ex.ctx = ctx; ex.dry = false; ex.mode = pl->d.mode; ex.eps = pl->d.eps;
    ex.stream = use_graph ? ctx->capture_stream : (cudaStream_t)stream;
    ex.q = pl->d.state_frac_bits ? ldexpf(1.f, -pl->d.state_frac_bits) : 0.f;
    ex.ws.dry = false; ex.ws.base = (char *)workspace; ex.ws.cap = pl->ws_bytes;
    if (ctx->profiling) ex.hold_ns = 5000000ull;     // the launches of a profiled step queue up behind a 5 ms hold
    if (use_graph) {
        if (pl->graph_exec) { cudaGraphExecDestroy(pl->graph_exec); pl->graph_exec = nullptr; }
        if (cudaStreamBeginCapture(ex.stream, cudaStreamCaptureModeRelaxed) != cudaSuccess)
            return fail(ctx, REVNET_E_CUDA, std::string("revnet_train_step: begin capture: ") + cudaGetErrorString(cudaGetLastError()));
    }
    float *recon = nullptr;
    revnet_step_stats local_stats;
    run_step(pl, ex, images, labels, params, grads, momentum, (char *)activations, loss, pred, logits, &local_stats, &recon);
    if (use_graph) {
        cudaGraph_t graph = nullptr;
        cudaError_t e = cudaStreamEndCapture(ex.stream, &graph);
        if (e != cudaSuccess || ex.failed || ex.ws.overflow) {
            if (graph) cudaGraphDestroy(graph);
            cudaGetLastError();
            if (ex.ws.overflow) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_train_step: workspace smaller than planned");
            if (!ex.failed) ctx->err = std::string("revnet_train_step: end capture: ") + cudaGetErrorString(e);
            return REVNET_E_CUDA;
        }
        e = cudaGraphInstantiate(&pl->graph_exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) { pl->graph_exec = nullptr; return fail(ctx, REVNET_E_CUDA, std::string("revnet_train_step: instantiate: ") + cudaGetErrorString(e)); }
        memcpy(pl->graph_key, key, sizeof key);
        pl->graph_stamping = ctx->stamping;
        pl->graph_stats = local_stats;
        if (cudaGraphLaunch(pl->graph_exec, (cudaStream_t)stream) != cudaSuccess)
            return fail(ctx, REVNET_E_CUDA, std::string("revnet_train_step: graph launch: ") + cudaGetErrorString(cudaGetLastError()));
        if (stats) *stats = local_stats;
        return REVNET_OK;
    }
    if (stats) *stats = local_stats;
    if (ex.ws.overflow) return fail(ctx, REVNET_E_WORKSPACE_TOO_SMALL, "revnet_train_step: workspace smaller than planned");
    if (ex.failed) return REVNET_E_CUDA;
    if (pl->d.verify_reconstruction && stats) {
        if (cudaMemcpyAsync(stats->recon_max_abs, recon, sizeof(float) * REVNET_MAX_STAGES, cudaMemcpyDeviceToHost, ex.stream) != cudaSuccess ||
            cudaStreamSynchronize(ex.stream) != cudaSuccess)
            return fail(ctx, REVNET_E_CUDA, std::string("revnet_train_step: ") + cudaGetErrorString(cudaGetLastError()));
        stats->device_status = read_device_status(ctx, ex.stream);      // the stream is idle here: the word is final for this step
    }
    return REVNET_OK;
}

extern "C" int revnet_train_step_host(revnet_ctx *ctx, revnet_plan *pl, const float *images_host, const int32_t *labels_host,
                                      float *images_dev, int32_t *labels_dev, float *params, float *grads, float *momentum,
                                      void *activations, void *workspace, float *loss_dev, int32_t *pred_dev,
                                      float *loss_host, int32_t *pred_host, revnet_step_stats *stats, void *stream) {
    if (!ctx || !pl || !images_host || !labels_host || !images_dev || !labels_dev || !loss_host || !pred_host)
        return fail(ctx, REVNET_E_INVALID_ARG, "revnet_train_step_host: null argument");
    cudaStream_t s = (cudaStream_t)stream;
    const revnet_stack_desc &d = pl->d;
    size_t ib = (size_t)d.N * d.img * d.img * d.in_ch * sizeof(float);
    if (cudaMemcpyAsync(images_dev, images_host, ib, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(labels_dev, labels_host, (size_t)d.N * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return fail(ctx, REVNET_E_CUDA, std::string("revnet_train_step_host: H2D copy: ") + cudaGetErrorString(cudaGetLastError()));
    int rc = revnet_train_step(ctx, pl, images_dev, labels_dev, params, grads, momentum, activations, workspace,
                               loss_dev, pred_dev, nullptr, stats, stream);
    if (rc) return rc;
    if (cudaMemcpyAsync(loss_host, loss_dev, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(pred_host, pred_dev, (size_t)d.N * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return fail(ctx, REVNET_E_CUDA, std::string("revnet_train_step_host: D2H copy: ") + cudaGetErrorString(cudaGetLastError()));
    // this call has synchronised: report what the step's kernels recorded (revnet_check_device clears it)
    const int st = read_device_status(ctx, s);
    if (stats) stats->device_status = st;
    if (st) return fail(ctx, st, "revnet_train_step_host: a kernel of the step recorded device status " + std::to_string(st));
    return REVNET_OK;
}
