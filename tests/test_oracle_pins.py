"""Pins for the CPU oracle: what the paper and the mathematics fix, never the oracle itself.

Each test would fail for a plausible slip in the oracle (dropped term, wrong sign or index,
transposed operand).  Sources: Section 2.2 Eq. 2 (BN-ReLU-conv), Section 3.1 (block and inverse),
Eq. 8 + Algorithm 1 (reconstructing backprop equals ordinary backprop), Section 3.2 (storage
independent of depth; 4N vs 3N cost).
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

from oracle import revnet as orc
from paper_1707_04585_b200 import synthetic as syn
from tests import helpers as hp

rng = np.random.default_rng(1234)


# ------------------------------------------------------------------ convolution and its adjoints
def brute_conv(a, w, s, p):
    N, Ci, H, W = a.shape
    Co, _, k, _ = w.shape
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    out = np.zeros((N, Co, Ho, Wo))
    for n in range(N):
        for co in range(Co):
            for i in range(Ho):
                for j in range(Wo):
                    acc = 0.0
                    for ci in range(Ci):
                        for kh in range(k):
                            for kw in range(k):
                                y, x = i * s + kh - p, j * s + kw - p
                                if 0 <= y < H and 0 <= x < W:
                                    acc += w[co, ci, kh, kw] * a[n, ci, y, x]
                    out[n, co, i, j] = acc
    return out


@pytest.mark.parametrize("k,s,p,H,W", [(3, 1, 1, 5, 6), (1, 1, 0, 4, 4), (3, 2, 1, 8, 6), (7, 2, 3, 12, 10), (3, 2, 1, 7, 5)])
def test_conv_matches_bruteforce_and_library(k, s, p, H, W):
    a = rng.standard_normal((2, 3, H, W))
    w = rng.standard_normal((4, 3, k, k))
    out = orc.conv_fwd(a, w, stride=s, pad=p)
    assert np.allclose(out, brute_conv(a, w, s, p), atol=1e-12)
    ta = torch.tensor(a, requires_grad=True)
    tw = torch.tensor(w, requires_grad=True)
    to = TF.conv2d(ta, tw, stride=s, padding=p)
    assert np.allclose(out, to.detach().numpy(), atol=1e-12)
    g = rng.standard_normal(out.shape)
    to.backward(torch.tensor(g))
    assert np.allclose(orc.conv_dgrad(g, w, (H, W), stride=s, pad=p), ta.grad.numpy(), atol=1e-12)
    assert np.allclose(orc.conv_wgrad(g, a, k, stride=s, pad=p), tw.grad.numpy(), atol=1e-11)


def test_conv_adjoint_identities():
    a = rng.standard_normal((2, 5, 6, 7)); w = rng.standard_normal((3, 5, 3, 3))
    g = rng.standard_normal((2, 3, 3, 4))
    lhs = float((orc.conv_fwd(a, w, stride=2) * g).sum())
    assert abs(lhs - float((a * orc.conv_dgrad(g, w, (6, 7), stride=2)).sum())) < 1e-10
    assert abs(lhs - float((w * orc.conv_wgrad(g, a, 3, stride=2)).sum())) < 1e-10


def test_conv_is_cross_correlation_not_flipped():
    a = np.zeros((1, 1, 5, 5)); a[0, 0, 2, 2] = 1.0
    w = np.arange(9.0).reshape(1, 1, 3, 3)
    out = orc.conv_fwd(a, w)
    # a unit impulse under cross-correlation returns the kernel mirrored about the centre
    assert np.array_equal(out[0, 0, 1:4, 1:4], w[0, 0, ::-1, ::-1])


def test_maxpool_library_and_first_max_tiebreak():
    a = rng.standard_normal((2, 3, 9, 8))
    out, idx = orc.maxpool_fwd(a)
    ta = torch.tensor(a, requires_grad=True)
    to = TF.max_pool2d(ta, 3, 2, 1)
    assert np.array_equal(out, to.detach().numpy())
    g = rng.standard_normal(out.shape)
    to.backward(torch.tensor(g))
    assert np.allclose(orc.maxpool_bwd(g, idx, (9, 8)), ta.grad.numpy())
    const = np.ones((1, 1, 4, 4))
    _, idx = orc.maxpool_fwd(const)
    assert idx[0, 0, 0, 0] == 0 and idx[0, 0, 1, 1] == 1 * 4 + 1   # first in row-major scan


# ------------------------------------------------------------------ BN + ReLU
def test_bn_relu_statistics_and_library():
    t = rng.standard_normal((6, 4, 5, 5)) * 3 + 1.5
    gamma = rng.standard_normal(4); beta = rng.standard_normal(4); eps = 1e-5
    a, (xhat, r, mask, _) = orc.bn_relu_fwd(t, gamma, beta, eps)
    var = t.var(axis=(0, 2, 3))
    assert np.allclose(xhat.mean(axis=(0, 2, 3)), 0, atol=1e-13)
    assert np.allclose(xhat.var(axis=(0, 2, 3)), var / (var + eps), rtol=1e-12)
    tt = torch.tensor(t, requires_grad=True)
    tg = torch.tensor(gamma, requires_grad=True); tb = torch.tensor(beta, requires_grad=True)
    ta = TF.relu(TF.batch_norm(tt, None, None, tg, tb, training=True, eps=eps))
    assert np.allclose(a, ta.detach().numpy(), atol=1e-12)
    da = rng.standard_normal(a.shape)
    ta.backward(torch.tensor(da))
    dt, dg, db = orc.bn_relu_bwd(da, (xhat, r, mask, gamma))
    assert np.allclose(dt, tt.grad.numpy(), atol=1e-12)
    assert np.allclose(dg, tg.grad.numpy(), atol=1e-12) and np.allclose(db, tb.grad.numpy(), atol=1e-12)
    # gradient through batch statistics is orthogonal to constants and to xhat, per channel
    assert np.allclose(dt.sum(axis=(0, 2, 3)), 0, atol=1e-12)
    # ... and to xhat up to the eps regulariser: sum(dt*xhat) = gamma r dgamma eps/(var+eps)
    expect = gamma * r.ravel() * dg * eps / (var + eps)
    assert np.allclose((dt * xhat).sum(axis=(0, 2, 3)), expect, atol=1e-12)


def test_bn_relu_scale_invariance():
    t = rng.standard_normal((8, 3, 4, 4))
    g = np.ones(3); b = np.zeros(3)
    a1, _ = orc.bn_relu_fwd(t, g, b, 0.0 + 1e-30)
    a2, _ = orc.bn_relu_fwd(7.5 * t + 2.0, g, b, 0.0 + 1e-30)
    assert np.allclose(a1, a2, atol=1e-10)


# ------------------------------------------------------------------ reversible block
def _block(kind="basic", c=4, w=2, N=3, H=5, W=4, seed=5):
    b = syn.BlockCfg(N, H, W, c, w, kind, seed)
    inp = syn.make_block_inputs(b, affine_jitter=True)
    F, G = hp.oracle_block(b, inp["params"])
    f64 = lambda k: inp[k].astype(np.float64)
    return b, inp, F, G, f64("x1"), f64("x2"), f64("dy1"), f64("dy2")


@pytest.mark.parametrize("kind", ["single", "basic", "bottleneck"])
def test_block_invertible_to_1e12(kind):
    b, inp, F, G, x1, x2, *_ = _block(kind)
    y1, y2 = orc.block_fwd(x1, x2, F, G, b.eps)
    r1, r2 = orc.block_inverse(y1, y2, F, G, b.eps)
    assert np.abs(r1 - x1).max() <= 1e-12 and np.abs(r2 - x2).max() <= 1e-12
    assert np.abs(y1 - x1).max() > 1e-3      # the block is not the identity


def test_block_special_cases():
    b, inp, F, G, x1, x2, *_ = _block("basic")
    zero = lambda fn: [dict(L, W=np.zeros_like(L["W"])) for L in fn]
    y1, y2 = orc.block_fwd(x1, x2, zero(F), zero(G), b.eps)
    assert np.array_equal(y1, x1) and np.array_equal(y2, x2)          # F = G = 0: identity
    y1, y2 = orc.block_fwd(x1, x2, F, zero(G), b.eps)
    assert np.array_equal(y2, x2) and not np.array_equal(y1, x1)      # G = 0: additive coupling on x1 only
    f, _ = orc.fn_fwd(x2, F, b.eps)
    assert np.allclose(y1 - x1, f, atol=1e-14)


@pytest.mark.parametrize("kind", ["single", "basic", "bottleneck"])
def test_algorithm1_equals_stored_backprop(kind):
    b, inp, F, G, x1, x2, dy1, dy2 = _block(kind)
    y1, y2, caches = orc.block_fwd(x1, x2, F, G, b.eps, keep=True)
    gs, gr = {}, {}
    sx1, sx2 = orc.block_bwd_stored(dy1, dy2, caches, gs)
    rx1, rx2, rdx1, rdx2 = orc.block_bwd_reconstruct(y1, y2, dy1, dy2, F, G, b.eps, gr)
    assert np.abs(rx1 - x1).max() <= 1e-12 and np.abs(rx2 - x2).max() <= 1e-12
    assert hp.rel_l2(rdx1, sx1) < 1e-10 and hp.rel_l2(rdx2, sx2) < 1e-10
    assert set(gs) == set(gr) and len(gs) == 3 * 2 * len(F)
    for k in gs:
        assert hp.rel_l2(gr[k], gs[k]) < 1e-10, k
    v1 = np.concatenate([gs[k].ravel() for k in sorted(gs)]); v2 = np.concatenate([gr[k].ravel() for k in sorted(gr)])
    cosang = float(v1 @ v2 / (np.linalg.norm(v1) * np.linalg.norm(v2)))
    assert math.degrees(math.acos(min(1.0, cosang))) < 1e-4


@pytest.mark.parametrize("kind", ["single", "basic", "bottleneck"])
def test_block_gradients_match_central_differences(kind):
    b, inp, F, G, x1, x2, dy1, dy2 = _block(kind, N=2, H=3, W=3, c=2, w=2)
    p64 = {k: v.astype(np.float64) for k, v in inp["params"].items()}

    def loss(x1_, x2_, params):
        F_, G_ = hp.oracle_block(b, params)
        y1, y2 = orc.block_fwd(x1_, x2_, F_, G_, b.eps)
        return float((y1 * dy1).sum() + (y2 * dy2).sum())

    F64, G64 = hp.oracle_block(b, p64)
    y1, y2 = orc.block_fwd(x1, x2, F64, G64, b.eps)
    grads = {}
    _, _, dx1, dx2 = orc.block_bwd_reconstruct(y1, y2, dy1, dy2, F64, G64, b.eps, grads)
    h = 1e-5
    checks = [("x1", dx1), ("x2", dx2)] + [(k, grads[k]) for k in grads]
    for name, g in checks:
        flat = g.ravel()
        for idx in rng.choice(flat.size, size=min(6, flat.size), replace=False):
            def shifted(d):
                if name == "x1":
                    t = x1.copy(); t.ravel()[idx] += d; return loss(t, x2, p64)
                if name == "x2":
                    t = x2.copy(); t.ravel()[idx] += d; return loss(x1, t, p64)
                q = dict(p64); t = p64[name].copy(); t.ravel()[idx] += d; q[name] = t
                return loss(x1, x2, q)
            fd = (shifted(h) - shifted(-h)) / (2 * h)
            assert abs(fd - flat[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, flat[idx])


# ------------------------------------------------------------------ stack
def torch_stack_grads(cfg, inp, taps=None):
    """Independent route: the same network written with library ops and differentiated by autograd.
    taps (a dict) receives the tensors between the layers -- ("x"|"y", stage, unit) -> (t1, t2) with
    their gradients retained, ("T", stage) -> (input, output) of a stored transition."""
    P = {k: torch.tensor(v.astype(np.float64), requires_grad=True) for k, v in inp["params"].items()}
    bnrc = lambda t, pre, s=1: TF.conv2d(TF.relu(TF.batch_norm(t, None, None, P[pre + ".gamma"], P[pre + ".beta"],
                                                               training=True, eps=cfg.eps)),
                                         P[pre + ".W"], stride=s, padding=P[pre + ".W"].shape[-1] // 2)
    h = TF.conv2d(torch.tensor(inp["images"].astype(np.float64)), P["stem.W"], stride=cfg.stem_stride, padding=cfg.stem_pad)
    if cfg.maxpool:
        h = TF.max_pool2d(h, 3, 2, 1)
    for si, s in enumerate(cfg.stages):
        if s.trans_k:
            hin = h
            h = bnrc(h, f"s{si}.T", s.trans_stride)
            if taps is not None:
                hin.retain_grad(); h.retain_grad()
                taps[("T", si)] = (hin, h)
        if s.down:
            # paper-shaped stage entry: y1 = S(x1) + F(x2), y2 = S(x2) + G(y1), S = 2x2 average pool + zero channels
            cp = h.shape[1] // 2
            S = lambda t: TF.pad(TF.avg_pool2d(t, 2, 2), (0, 0, 0, 0, 0, s.c - cp))
            f = h[:, cp:]
            for li, ly in enumerate(syn.down_fn_layers(s.kind, cp, s.c, s.w)):
                f = bnrc(f, f"s{si}.d.F.l{li}", ly[3])
            y1 = S(h[:, :cp]) + f
            g = y1
            for li in range(len(syn.fn_layers(s.kind, s.c, s.w))):
                g = bnrc(g, f"s{si}.d.G.l{li}")
            h = torch.cat([y1, S(h[:, cp:]) + g], dim=1)
        x1, x2 = h[:, :s.c], h[:, s.c:]
        nl = len(syn.fn_layers(s.kind, s.c, s.w))
        for u in range(syn.reversible_units(s)):
            if taps is not None:
                x1, x2 = x1 * 1.0, x2 * 1.0           # fresh nodes, so that each unit's input gradient can be read
                x1.retain_grad(); x2.retain_grad()
                taps[("x", si, u)] = (x1, x2)
            f = x2
            for li in range(nl):
                f = bnrc(f, f"s{si}.u{u}.F.l{li}")
            x1 = x1 + f
            g = x1
            for li in range(nl):
                g = bnrc(g, f"s{si}.u{u}.G.l{li}")
            x2 = x2 + g
            if taps is not None:
                x1.retain_grad(); x2.retain_grad()
                taps[("y", si, u)] = (x1, x2)
        h = torch.cat([x1, x2], dim=1)
    logits = h.mean(dim=(2, 3)) @ P["fc.W"].T + P["fc.b"]
    loss = TF.cross_entropy(logits, torch.tensor(inp["labels"].astype(np.int64)))
    loss.backward()
    return logits.detach().numpy(), float(loss.detach()), {k: v.grad.numpy() for k, v in P.items()}


@pytest.mark.parametrize("kind,maxpool", [("basic", False), ("bottleneck", False), ("bottleneck", True)])
def test_stack_against_autograd_and_reconstruct_equals_stored(kind, maxpool):
    cfg = hp.tiny_stack(kind, maxpool)
    inp = syn.make_stack_inputs(cfg, affine_jitter=True)
    net = hp.oracle_net(cfg, inp["params"])
    rs = orc.stack_train_grads(net, inp["images"], inp["labels"], "stored")
    rr = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct")
    tl, tloss, tg = torch_stack_grads(cfg, inp)
    assert np.allclose(rs["logits"], tl, atol=1e-10) and abs(rs["loss"] - tloss) < 1e-12
    assert set(tg) == set(rs["grads"]) == set(rr["grads"])
    for k in tg:
        assert hp.rel_l2(rs["grads"][k], tg[k]) < 1e-9, k
        assert hp.rel_l2(rr["grads"][k], rs["grads"][k]) < 1e-9, k
    for key, (x1, x2) in rr["recovered"].items():
        f1, f2 = rr["block_inputs"][key]
        assert np.abs(x1 - f1).max() < 1e-11 and np.abs(x2 - f2).max() < 1e-11
    assert np.array_equal(rs["pred"], tl.argmax(axis=1))


def test_per_block_records_inside_a_stack_match_autograd():
    """The (y1,y2,dy1,dy2) -> (dx1,dx2) the oracle reports for single blocks and transitions inside a
    network equal what autograd sees at the same places (Section 3.2: Algorithm 1 applied block by block)."""
    cfg = hp.tiny_stack("bottleneck", True, units=3)
    inp = syn.make_stack_inputs(cfg, affine_jitter=True)
    net = hp.oracle_net(cfg, inp["params"])
    keys = {(0, 0), (0, 2), (1, 1)}
    rr = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct", keep_blocks=keys, keep_transitions=True)
    taps = {}
    torch_stack_grads(cfg, inp, taps)
    assert set(rr["blocks"]) == keys
    for (si, u), b in rr["blocks"].items():
        (x1, x2), (y1, y2) = taps[("x", si, u)], taps[("y", si, u)]
        for got, ref in ((b["y1"], y1.detach()), (b["y2"], y2.detach()), (b["dy2"], y2.grad), (b["dx1"], x1.grad), (b["dx2"], x2.grad)):
            assert hp.rel_l2(got, ref.numpy()) < 1e-9, (si, u)
        # y1 feeds G as well as the next layer: the gradient Algorithm 1 is handed for it is the direct part only
        # (autograd's total minus G's share), i.e. dx1 = dy1 + (dG/dy1)^T dy2  =>  check through dx1 above and here
        g = {}
        F, G = net["stages"][si]["units"][u]
        _, _, d1, d2 = orc.block_bwd_reconstruct(b["y1"], b["y2"], b["dy1"], b["dy2"], F, G, net["eps"], g)
        assert hp.rel_l2(d1, b["dx1"]) < 1e-12 and hp.rel_l2(d2, b["dx2"]) < 1e-12
        for k, v in g.items():
            assert hp.rel_l2(v, rr["grads"][k]) < 1e-12, k
    for si, t in rr["transitions"].items():
        hin, hout = taps[("T", si)]
        assert hp.rel_l2(t["x"], hin.detach().numpy()) < 1e-10
        assert hp.rel_l2(t["dy"], hout.grad.numpy()) < 1e-9 and hp.rel_l2(t["dx"], hin.grad.numpy()) < 1e-9


def paper_tiny(kind):
    """A small network shaped like the paper's table: no separate transitions, the first unit of stages 2.. down-samples."""
    if kind == "basic":
        st = (syn.StageCfg(2, 4, 0, "basic", 0, 1), syn.StageCfg(2, 8, 0, "basic", 0, 1, down=True), syn.StageCfg(1, 12, 0, "basic", 0, 1, down=True))
    else:
        st = (syn.StageCfg(1, 8, 4, "bottleneck", 3, 1), syn.StageCfg(2, 16, 4, "bottleneck", 0, 1, down=True))
    return syn.StackCfg(f"paper_tiny_{kind}", 4, 16, 5, 3, 1, 8, False, st, seed=17)


def test_shortcut_is_average_pool_plus_zero_channels_and_its_adjoint():
    x = rng.standard_normal((2, 3, 6, 4)); d = rng.standard_normal((2, 5, 3, 2))
    y = orc.shortcut_fwd(x, 5)
    assert np.allclose(y[:, :3], TF.avg_pool2d(torch.tensor(x), 2, 2).numpy(), atol=1e-14) and np.all(y[:, 3:] == 0)
    assert abs((y * d).sum() - (x * orc.shortcut_bwd(d, 3)).sum()) < 1e-12          # <S x, d> = <x, S^T d>


@pytest.mark.parametrize("kind", ["basic", "bottleneck"])
def test_paper_shaped_stack_against_autograd(kind):
    """Down-sampling inside the first unit of a stage (Table "Architectural details"): the stack with such units
    against the same network written with library ops; both backward flavours agree; a fixed-point state still
    reconstructs every reversible unit's input exactly."""
    cfg = paper_tiny(kind)
    inp = syn.make_stack_inputs(cfg, affine_jitter=True)
    net = hp.oracle_net(cfg, inp["params"])
    rs = orc.stack_train_grads(net, inp["images"], inp["labels"], "stored")
    rr = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct")
    tl, tloss, tg = torch_stack_grads(cfg, inp)
    assert np.allclose(rs["logits"], tl, atol=1e-10) and abs(rs["loss"] - tloss) < 1e-12
    assert set(tg) == set(rs["grads"]) == set(rr["grads"])
    for k in tg:
        assert hp.rel_l2(rs["grads"][k], tg[k]) < 1e-9, k
        assert hp.rel_l2(rr["grads"][k], rs["grads"][k]) < 1e-9, k
    num = {"bf16_operands": True, "frac_bits": 16}
    rq = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct", num=num)
    for key, (x1, x2) in rq["block_inputs"].items():
        assert np.array_equal(rq["recovered"][key][0], x1) and np.array_equal(rq["recovered"][key][1], x2), key


def test_paper_table_parameter_counts_all_rows():
    """All four RevNet rows of the table, counted on the paper-shaped configurations (every parameter: conv, BN, FC)."""
    rows = {}
    with open(__file__.replace("test_oracle_pins.py", "golden/arch_table.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, bott, units, ch, pm = line.split()
                rows[name] = ([int(u) for u in units.split("-")], float(pm))
    tol = {"RevNet-38": 0.02, "RevNet-110": 0.02, "RevNet-164": 0.04, "RevNet-104": 0.10}
    for name, (units, pm) in rows.items():
        cfg = syn.stack_config("paper_" + name.lower().replace("-", ""))
        assert [s.units for s in cfg.stages] == units
        assert all(s.down for s in cfg.stages[1:]) and not any(s.trans_k for s in cfg.stages[1:])
        n = sum(int(np.prod(shape)) for _, shape, _ in syn.param_specs(cfg))
        assert abs(n / 1e6 - pm) / pm < tol[name], (name, n)


def test_storage_flat_in_depth_and_cost_4n_vs_3n():
    sizes, ratio = {}, {}
    for units in (1, 2, 5):
        cfg = hp.tiny_stack("basic", units=units)
        inp = syn.make_stack_inputs(cfg)
        net = hp.oracle_net(cfg, inp["params"])
        for mode in ("stored", "reconstruct"):
            orc.FLOPS["conv"] = 0
            r = orc.stack_train_grads(net, inp["images"], inp["labels"], mode)
            sizes[(units, mode)] = r["stored_bytes"]
            ratio[(units, mode)] = orc.FLOPS["conv"]
    assert sizes[(1, "reconstruct")] == sizes[(2, "reconstruct")] == sizes[(5, "reconstruct")]
    assert sizes[(1, "stored")] < sizes[(2, "stored")] < sizes[(5, "stored")]
    # cost of the reversible units alone: difference between depths isolates them (Section 3.2)
    d_rec = ratio[(5, "reconstruct")] - ratio[(2, "reconstruct")]
    d_sto = ratio[(5, "stored")] - ratio[(2, "stored")]
    assert d_rec * 3 == d_sto * 4


def test_head_closed_forms_and_sgd():
    loss, dl = orc.softmax_ce(np.zeros((4, 10)), np.array([1, 2, 3, 4]))
    assert abs(loss - math.log(10.0)) < 1e-15
    assert np.allclose(dl.sum(axis=1), 0) and abs(dl[0, 1] - (0.1 - 1) / 4) < 1e-15
    big, _ = orc.softmax_ce(np.array([[1000.0, 0.0]]), np.array([1]))
    assert abs(big - 1000.0) < 1e-9                                     # no overflow
    p = {"w": np.array([1.0, -2.0]), "g": np.array([0.5])}
    g = {"w": np.array([0.1, 0.2]), "g": np.array([1.0])}
    v = {"w": np.array([1.0, 1.0]), "g": np.array([0.0])}
    np_, nv = orc.sgd_step(p, g, v, lr=0.1, momentum=0.9, weight_decay=0.5, decayed={"w"})
    assert np.allclose(nv["w"], [0.9 + 0.1 + 0.5, 0.9 + 0.2 - 1.0]) and np.allclose(nv["g"], [1.0])
    assert np.allclose(np_["w"], [1.0 - 0.15, -2.0 - 0.01]) and np.allclose(np_["g"], [0.4])


def test_paper_table_parameter_counts():
    """Table "Architectural details": parameter counts of the RevNet rows.  Read with the
    down-sampling inside the first unit of a stage (the table's unit counts), conv + FC weights
    only; the printed figures are matched to a few percent."""
    rows = {}
    with open(__file__.replace("test_oracle_pins.py", "golden/arch_table.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, bott, units, ch, pm = line.split()
                rows[name] = (bott == "yes", [int(u) for u in units.split("-")], [int(c) for c in ch.split("-")], float(pm))

    def count(bott, units, ch, ncls, stem_k, per_half_w=None):
        total = 3 * ch[0] * stem_k ** 2
        cin = ch[0]
        for si, (u, ctot) in enumerate(zip(units, ch[1:])):
            c = ctot // 2
            for ui in range(u):
                cin_half = (cin // 2) if ui == 0 else c
                if not bott:
                    total += 2 * (cin_half * c * 9 + c * c * 9)
            cin = ctot
        return total + cin * ncls
    for name in ("RevNet-38", "RevNet-110"):
        bott, units, ch, pm = rows[name]
        n = count(bott, units, ch, 10, 3)
        assert abs(n / 1e6 - pm) / pm < 0.05, (name, n)
    # the benchmark configs use the same stage widths with separate stored transitions
    c38 = syn.stack_config("revnet38")
    assert [2 * s.c for s in c38.stages] == rows["RevNet-38"][2][1:]
    assert [s.units for s in c38.stages] == rows["RevNet-38"][1]
    c110 = syn.stack_config("revnet110")
    assert [2 * s.c for s in c110.stages] == rows["RevNet-110"][2][1:] and [s.units for s in c110.stages] == [9, 9, 9]
    assert [s.w for s in syn.stack_config("revnet104").stages] == rows["RevNet-104"][2]
