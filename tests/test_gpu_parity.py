"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Tolerances (relative L2 per tensor unless stated):
  strict fp32 mode : 1e-4 everywhere
  bf16 mode        : block outputs / logits 2e-2, gradients 5e-2
  reconstruction   : recovered x1, x2 within 1e-3 max-abs of the inputs that produced y1, y2;
                     on the fixed-point coupling state (the bf16 mode's default) they are bit-exact
  integers (arg-max predictions) : exact

Which comparisons are held to these numbers directly and which few (end-to-end gradients of deep
stacks) may use the oracle's measured self-sensitivity instead is decided per comparison by the
caller and recorded: see tests/parity.py.  Algorithm 1 is a per-block statement, so the deep
configurations are also checked block by block INSIDE the network: the oracle's (y1, y2, dy1, dy2)
of a unit go through revnet_block_bwd and every output is held to the stated tolerance.
"""
import numpy as np
import pytest
import torch

from oracle import revnet as orc
from paper_1707_04585_b200 import binding as B
from paper_1707_04585_b200 import runner as R
from paper_1707_04585_b200 import synthetic as syn
from tests import helpers as hp
from tests import parity as par

pytestmark = pytest.mark.gpu

TOL = par.TOL
RECON = par.RECON


def perturb_levels(runner):
    return [1e-6] + ([2.0 ** -runner.frac] if runner.frac else [])


def oracle_numerics(runner):
    """Storage roundings the oracle applies so that discrete decisions (ReLU sign, grid point of a
    stored value) are taken at the kernel's precision: bf16 conv operands in mode 0, the
    fixed-point grid of the coupling state when one is used.  Arithmetic stays float64."""
    num = {}
    if runner.mode == 0:
        num["bf16_operands"] = True
    if runner.frac:
        num["frac_bits"] = runner.frac
    return num or None


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    B.revnet_check_device(c)      # no kernel may have given up a bounded wait
    c.close()


def block_case_name(b, mode, extra=""):
    return f"block {b.kind} N{b.N} {b.H}x{b.W} c{b.c} w{b.w} mode{mode}{extra}"


def perturbed(rng, a, level, grid):
    """a * (1 + level * u), u uniform in [-1, 1], put back on the fixed-point grid if there is one."""
    p = a * (1 + level * rng.uniform(-1, 1, a.shape))
    return np.rint(p * grid) / grid if grid else p


FLOOR_DRAWS = 3      # perturbed oracle runs per level for small cases: a differing ReLU decision is a rare event, one draw may see none


def run_block_case(ctx, b, mode, jitter, inplace, tag=""):
    """One reversible block, forward and reconstructing backward.  Forward outputs and, for cases in
    which no ReLU decision is expected to differ (parity.block_floor_allowed), every gradient are
    held to the stated tolerance; the larger cases go by the floor rule."""
    inp = syn.make_block_inputs(b, affine_jitter=jitter)
    F, G = hp.oracle_block(b, inp["params"])
    r = R.BlockRunner(ctx, b, mode)
    r.load(inp["params"])
    num = oracle_numerics(r)
    x1, x2, dy1, dy2 = (inp[k].astype(np.float64) for k in ("x1", "x2", "dy1", "dy2"))
    grid = float(1 << r.frac) if r.frac else None
    if grid:
        x1, x2 = np.rint(x1 * grid) / grid, np.rint(x2 * grid) / grid
    case = block_case_name(b, mode, tag + (" inplace" if inplace else ""))
    t = TOL[mode]

    py1, py2 = orc.block_fwd(x1, x2, F, G, b.eps)                    # the plain float64 definition
    oy1, oy2 = orc.block_fwd(x1, x2, F, G, b.eps, num=num)
    og = {}
    _, _, odx1, odx2 = orc.block_bwd_reconstruct(oy1, oy2, dy1, dy2, F, G, b.eps, og, num=num)
    og["dx1"], og["dx2"] = odx1, odx2
    y1, y2 = r.forward(inp["x1"], inp["x2"], inplace=inplace)
    par.check(case + " fwd vs plain fp64", dict(y1=y1, y2=y2), dict(y1=py1, y2=py2), t["out"])
    par.check(case + " fwd", dict(y1=y1, y2=y2), dict(y1=oy1, y2=oy2), t["out"])
    # backward from the GPU's own outputs: reconstruction must return the inputs that produced them
    rx1, rx2, dx1, dx2, grads = r.backward(y1, y2, inp["dy1"], inp["dy2"], inplace=inplace)
    assert np.abs(rx1 - x1).max() <= RECON and np.abs(rx2 - x2).max() <= RECON
    if grid:        # fixed-point state: the inputs as the kernel saw them come back bit for bit
        assert np.array_equal(rx1, x1) and np.array_equal(rx2, x2)
    grads["dx1"], grads["dx2"] = dx1, dx2
    assert set(grads) == set(og)
    allow = ("*",) if par.block_floor_allowed(mode, b.N, b.H, b.W, syn.fn_layers(b.kind, b.c, b.w)) else ()

    def floor_fn():
        out = []
        for lv in perturb_levels(r):
            for draw in range(FLOOR_DRAWS):
                rng = np.random.default_rng(99 + draw)
                p1, p2 = perturbed(rng, x1, lv, grid), perturbed(rng, x2, lv, grid)
                q1, q2 = orc.block_fwd(p1, p2, F, G, b.eps, num=num)
                g_ = {}
                _, _, d1_, d2_ = orc.block_bwd_reconstruct(q1, q2, dy1, dy2, F, G, b.eps, g_, num=num)
                g_["dx1"], g_["dx2"] = d1_, d2_
                out.append(g_)
        return out
    return par.check(case + " bwd", grads, og, t["grad"], floor_fn, allow, floor_scope="case")


def test_config1_single_block_strict(ctx):
    """N=4, C=16 (8+8), 8x8, F and G = BN-ReLU-conv3x3, gamma=1, beta=0, seed 0, fp32."""
    run_block_case(ctx, syn.block_config_1(), mode=1, jitter=False, inplace=False)


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("kind,N,H,W,c,w", [
    ("single", 4, 8, 8, 8, 0),
    ("basic", 3, 5, 7, 12, 0),        # ragged: pixel count 105, channels not a power of two
    ("basic", 8, 32, 32, 16, 0),      # several tiles (8192 pixels)
    ("basic", 2, 16, 16, 56, 0),
    ("bottleneck", 2, 16, 16, 128, 32),
    ("bottleneck", 3, 7, 7, 64, 16),
    ("basic", 1, 1, 1, 4, 0),         # degenerate: one pixel
    ("basic", 3, 14, 14, 32, 0),      # image rows not a divisor of the 128-row tile: ragged last tile per image
    ("basic", 1, 28, 28, 16, 0),      # row pitch padded (28 -> 32 accumulator rows per image row)
    ("bottleneck", 2, 56, 56, 64, 16),  # large-image stage shape at reduced width: two image rows per tile
    ("basic", 5, 8, 8, 24, 0),        # channel count padded to 32; odd number of two-image tiles
    ("basic", 2, 8, 8, 40, 0),        # 40 channels: no single K chunk, the per-tap TMA kernel takes it
    ("bottleneck", 4, 8, 8, 96, 24),  # 1x1 convolutions with more than 64 input channels
])
@pytest.mark.parametrize("inplace", [False, True])
def test_block_parity(ctx, mode, kind, N, H, W, c, w, inplace):
    if N * H * W == 1:
        # a single pixel per channel has zero variance: BN output is beta, gradients through BN vanish
        b = syn.BlockCfg(N, H, W, c, w, kind, seed=7)
        inp = syn.make_block_inputs(b, affine_jitter=True)
        r = R.BlockRunner(ctx, b, mode); r.load(inp["params"])
        F, G = hp.oracle_block(b, inp["params"])
        oy1, oy2 = orc.block_fwd(inp["x1"].astype(np.float64), inp["x2"].astype(np.float64), F, G, b.eps)
        y1, y2 = r.forward(inp["x1"], inp["x2"], inplace=inplace)
        assert np.allclose(y1, oy1, atol=2e-2 if mode == 0 else 1e-4) and np.allclose(y2, oy2, atol=2e-2 if mode == 0 else 1e-4)
        return
    run_block_case(ctx, syn.BlockCfg(N, H, W, c, w, kind, seed=100 + c), mode, jitter=True, inplace=inplace)


def test_block_deterministic_and_recompute_bit_exact(ctx):
    """Same input twice -> identical bits; so the G(y1) recomputed in the backward equals the forward's."""
    b = syn.BlockCfg(4, 16, 16, 32, 0, "basic", seed=3)
    inp = syn.make_block_inputs(b, affine_jitter=True)
    for mode in (0, 1):
        r = R.BlockRunner(ctx, b, mode); r.load(inp["params"])
        a = r.forward(inp["x1"], inp["x2"]); c = r.forward(inp["x1"], inp["x2"])
        assert np.array_equal(a[0], c[0]) and np.array_equal(a[1], c[1])
        g1 = r.backward(a[0], a[1], inp["dy1"], inp["dy2"]); g2 = r.backward(a[0], a[1], inp["dy1"], inp["dy2"])
        for u, v in zip(g1[:4], g2[:4]):
            assert np.array_equal(u, v)
        for k in g1[4]:
            assert np.array_equal(g1[4][k], g2[4][k]), k


def test_reconstruction_drift_over_depth(ctx):
    """Chain 12 blocks forward in place, then reverse them: the recovered inputs of every block stay
    within 1e-3 max-abs of what the forward pass saw."""
    b = syn.BlockCfg(4, 16, 16, 16, 0, "basic", seed=21)
    runners, fw = [], []
    inp0 = syn.make_block_inputs(b)
    x1, x2 = inp0["x1"], inp0["x2"]
    for i in range(12):
        bi = syn.BlockCfg(b.N, b.H, b.W, b.c, b.w, b.kind, seed=200 + i)
        r = R.BlockRunner(ctx, bi, 0); r.load(syn.make_block_inputs(bi, affine_jitter=True)["params"])
        runners.append(r); fw.append((x1, x2))
        x1, x2 = r.forward(x1, x2, inplace=True)
    d1, d2 = inp0["dy1"], inp0["dy2"]
    worst = 0.0
    for r, (f1, f2) in zip(reversed(runners), reversed(fw)):
        x1, x2, d1, d2, _ = r.backward(x1, x2, d1, d2, inplace=True)
        worst = max(worst, np.abs(x1 - f1).max(), np.abs(x2 - f2).max())
    assert worst <= 2.0 ** -16, worst     # only the quantisation of the very first input


def test_float_state_strict_mode_reconstruction(ctx):
    """float32 coupling state with fp32 arithmetic: reconstruction error stays at rounding level."""
    b = syn.BlockCfg(4, 16, 16, 16, 0, "basic", seed=21)
    inp = syn.make_block_inputs(b, affine_jitter=True)
    r = R.BlockRunner(ctx, b, 1, frac_bits=0); r.load(inp["params"])
    y1, y2 = r.forward(inp["x1"], inp["x2"])
    x1, x2, *_ = r.backward(y1, y2, inp["dy1"], inp["dy2"])
    assert np.abs(x1 - inp["x1"]).max() <= 1e-5 and np.abs(x2 - inp["x2"]).max() <= 1e-5


ORACLE_RUNS = {}


def oracle_stack_run(cfg, inp, net, num, keep_blocks=(), keep_transitions=False, level=0.0, draw=0):
    """One oracle step, memoised for the session (several tests look at the same run)."""
    key = (cfg, repr(num), tuple(sorted(keep_blocks)), keep_transitions, level, draw)
    if key not in ORACLE_RUNS:
        images = inp["images"].astype(np.float64)
        if level:
            images = images * (1 + level * np.random.default_rng(98 + draw).uniform(-1, 1, images.shape))
        ORACLE_RUNS[key] = orc.stack_train_grads(net, images, inp["labels"], "reconstruct", num=num,
                                                 keep_blocks=keep_blocks, keep_transitions=keep_transitions)
    return ORACLE_RUNS[key]


def e2e_allow(cfg, mode):
    """End-to-end tensors of a whole train step that go by the floor rule (tests/parity.py): in the bf16 mode
    everything behind the classifier -- two or three layers in, the kernel's and the oracle's activations differ at
    the bf16 noise level, and from there on ReLU decisions differ in every layer, the top unit included.  In strict
    mode the same tensors of networks whose layers are large enough for fp32 rounding to flip a decision."""
    if mode == 0:
        return ("*",)
    res = syn.stage_resolutions(cfg)
    big = max(par.sign_decisions_expected_to_differ(cfg.N * H * H * max(s.c, s.w), 9 * max(s.c, s.w)) for s, H in zip(cfg.stages, res))
    return ("stem.*", "s*") if big >= 0.05 else ()


def run_stack_case(ctx, cfg, mode, jitter=True, plain_forward=False, floor_allowed=None, floor_levels=None,
                   keep_blocks=(), keep_transitions=False, logits_floor=False, floor_draws=FLOOR_DRAWS):
    """One whole train step against the oracle.  floor_allowed: gradient tensors that go by the floor rule (default:
    e2e_allow); logits_floor: the logits too (bf16 mode of the deep bottleneck networks only)."""
    if floor_allowed is None:
        floor_allowed = e2e_allow(cfg, mode)
    inp = syn.make_stack_inputs(cfg, affine_jitter=jitter)
    net = hp.oracle_net(cfg, inp["params"])
    r = R.StackRunner(ctx, cfg, mode, verify_reconstruction=True)
    num = oracle_numerics(r)
    o = oracle_stack_run(cfg, inp, net, num, keep_blocks, keep_transitions)
    zero_v = {k: np.zeros_like(v, dtype=np.float64) for k, v in inp["params"].items()}
    op, ov = orc.sgd_step(inp["params"], o["grads"], zero_v, cfg.lr, cfg.momentum, cfg.weight_decay, hp.decayed_names(cfg))
    r.load(inp["images"], inp["labels"], inp["params"])
    st = r.step()
    g = r.results()
    t = dict(TOL[mode])
    case = f"stack {cfg.name} N{cfg.N} mode{mode}"
    levels = perturb_levels(r) if floor_levels is None else floor_levels

    def floor_runs():
        return [oracle_stack_run(cfg, inp, net, num, level=lv, draw=dr) for lv in levels for dr in range(floor_draws)]

    # forward quantities: the stated tolerance, except where the caller said beforehand that the depth of the network
    # lets bf16 rounding differences grow beyond it
    _, lfloor = par.check(case + " logits", dict(logits=g["logits"]), dict(logits=o["logits"]), t["out"],
                          lambda: [dict(logits=f["logits"]) for f in floor_runs()], ("logits",) if logits_floor else ())
    if plain_forward:       # also against the unrounded float64 definition
        plain = oracle_stack_run(cfg, inp, net, None)
        par.check(case + " logits vs plain fp64", dict(logits=g["logits"]), dict(logits=plain["logits"]), t["out"])
    assert abs(g["loss"] - o["loss"]) <= max(t["out"], par.FLOOR_FACTOR * lfloor) * max(1.0, abs(o["loss"]))
    # arg-max: the kernel must agree exactly with the arg-max of its own logits, and with the oracle
    # wherever the oracle's top-2 margin exceeds the logit tolerance
    assert np.array_equal(g["pred"], g["logits"].argmax(axis=1).astype(np.int32))
    srt = np.sort(o["logits"], axis=1)
    margin = srt[:, -1] - srt[:, -2]
    clear = margin > 2 * max(t["out"], par.FLOOR_FACTOR * lfloor) * np.abs(o["logits"]).max()
    assert np.array_equal(g["pred"][clear], o["pred"][clear])
    if mode == 1:
        assert np.array_equal(g["pred"], o["pred"])
    worst, floor = par.check(case + " grads", g["grads"], o["grads"], t["grad"],
                             lambda: [f["grads"] for f in floor_runs()], floor_allowed)
    # momentum = gradient + weight decay (same rule as the gradient it comes from); the updated weights
    # move by lr * momentum, a small part of their norm: stated tolerance
    fl_mom = None
    if floor_allowed:
        def fl_mom():
            out = []
            for f in floor_runs():
                out.append(orc.sgd_step(inp["params"], f["grads"], zero_v, cfg.lr, cfg.momentum, cfg.weight_decay, hp.decayed_names(cfg))[1])
            return out
    par.check(case + " momentum", g["momentum"], ov, t["grad"], fl_mom, floor_allowed)
    # updated weights: w - lr * momentum.  For weights the step is a small part of the norm; BN shifts start at zero,
    # so their updated value IS the step: same rule as the gradients
    fl_par = None
    if floor_allowed:
        def fl_par():
            return [orc.sgd_step(inp["params"], f["grads"], zero_v, cfg.lr, cfg.momentum, cfg.weight_decay, hp.decayed_names(cfg))[0] for f in floor_runs()]
    par.check(case + " updated params", g["params"], op, t["grad"], fl_par, floor_allowed)
    for si in range(len(cfg.stages)):
        assert st.recon_max_abs[si] <= RECON, (si, st.recon_max_abs[si])
        if r.frac:
            assert st.recon_max_abs[si] == 0.0, (si, st.recon_max_abs[si])   # fixed-point state: exact
    assert st.stored_activation_bytes == o["stored_bytes"]
    return st, worst, floor


def run_blocks_in_network(ctx, cfg, mode, keys, jitter=False):
    """Algorithm 1 block by block inside a full network: the oracle's (y1, y2, dy1, dy2) of a unit go
    through revnet_block_bwd; x1, x2 within 1e-3 max-abs and dx1, dx2, dW, dgamma, dbeta within the
    stated tolerance.  One block does not accumulate rounding decisions the way a whole stack does.
    Likewise every stored transition through revnet_transition_fwd / _bwd."""
    inp = syn.make_stack_inputs(cfg, affine_jitter=jitter)
    net = hp.oracle_net(cfg, inp["params"])
    frac = R.DEFAULT_FRAC_BITS[mode]
    num = {}
    if mode == 0: num["bf16_operands"] = True
    if frac: num["frac_bits"] = frac
    num = num or None
    o = oracle_stack_run(cfg, inp, net, num, tuple(sorted(keys)), True)
    res = syn.stage_resolutions(cfg)
    t = TOL[mode]
    for (si, u) in sorted(keys):
        s = cfg.stages[si]
        rec = o["blocks"][(si, u)]
        b = syn.BlockCfg(cfg.N, res[si], res[si], s.c, s.w, s.kind, seed=0, eps=cfg.eps)
        params = {k[len(f"s{si}.u{u}."):]: v for k, v in inp["params"].items() if k.startswith(f"s{si}.u{u}.")}
        r = R.BlockRunner(ctx, b, mode)
        r.load(params)
        rx1, rx2, dx1, dx2, grads = r.backward(rec["y1"], rec["y2"], rec["dy1"].astype(np.float32), rec["dy2"].astype(np.float32), inplace=True)
        # the inputs rebuilt from the ORACLE's outputs differ from the oracle's inputs by what the kernel's F and G
        # differ from the oracle's: the block-output tolerance (exact inversion is asserted where the kernel's own
        # outputs are reversed)
        fx1, fx2 = o["block_inputs"][(si, u)]
        par.check(f"in-network block {cfg.name} N{cfg.N} s{si}.u{u} mode{mode} rebuilt inputs", dict(x1=rx1, x2=rx2), dict(x1=fx1, x2=fx2), t["out"])
        got = dict(grads)
        got["dx1"], got["dx2"] = dx1, dx2
        ref = {k: o["grads"][f"s{si}.u{u}.{k}"] for k in grads}
        ref["dx1"], ref["dx2"] = rec["dx1"], rec["dx2"]
        allow = ("*",) if par.block_floor_allowed(mode, b.N, b.H, b.W, syn.fn_layers(b.kind, b.c, b.w)) else ()
        F, G = net["stages"][si]["units"][u]
        grid = float(1 << frac) if frac else None

        def floor_fn(rec=rec, F=F, G=G, grid=grid, si=si, u=u):
            out = []
            pre = f"s{si}.u{u}."
            for lv in ([1e-6] + ([2.0 ** -frac] if frac else [])):
                for draw in range(FLOOR_DRAWS):
                    rng = np.random.default_rng(97 + draw)
                    p1, p2 = perturbed(rng, rec["y1"], lv, grid), perturbed(rng, rec["y2"], lv, grid)
                    g_ = {}
                    _, _, d1_, d2_ = orc.block_bwd_reconstruct(p1, p2, rec["dy1"], rec["dy2"], F, G, cfg.eps, g_, num=num)
                    g_ = {k[len(pre):]: v for k, v in g_.items()}
                    g_["dx1"], g_["dx2"] = d1_, d2_
                    out.append(g_)
            return out
        par.check(f"in-network block {cfg.name} N{cfg.N} s{si}.u{u} mode{mode}", got, ref, t["grad"], floor_fn, allow, floor_scope="case")
    for si, s in enumerate(cfg.stages):
        if s.trans_k:
            rec = o["transitions"][si]
            got = transition_through_abi(ctx, rec["x"], rec["dy"], inp["params"][f"s{si}.T.W"], inp["params"][f"s{si}.T.gamma"],
                                         inp["params"][f"s{si}.T.beta"], s.trans_stride, si > 0, mode, frac, cfg.eps)
            ref = {"dx": rec["dx"], f"s{si}.T.W": o["grads"][f"s{si}.T.W"], f"s{si}.T.gamma": o["grads"][f"s{si}.T.gamma"],
                   f"s{si}.T.beta": o["grads"][f"s{si}.T.beta"]}
            x1n, x2n = o["block_inputs"][(si, 0)]
            par.check(f"in-network transition {cfg.name} N{cfg.N} s{si}.T mode{mode} fwd", dict(y=got["y"]),
                      dict(y=np.concatenate([x1n, x2n], axis=1)), 1e-4 if mode else 2e-3)
            par.check(f"in-network transition {cfg.name} N{cfg.N} s{si}.T mode{mode} bwd",
                      {"dx": got["dx"], f"s{si}.T.W": got["dW"], f"s{si}.T.gamma": got["dgamma"], f"s{si}.T.beta": got["dbeta"]}, ref, t["grad"])
    return o


def transition_through_abi(ctx, x, dy, W, gamma, beta, stride, split, mode, frac, eps):
    """BN -> ReLU -> conv of a stored layer, forward and backward, through revnet_transition_*.
    x [N,cin,H,H], dy [N,cout,Ho,Ho] float64 NCHW; split: x is the (x1,x2) pair of a coupling state."""
    N, cin, H, _ = x.shape
    cout, _, k, _ = W.shape
    Ho = dy.shape[2]
    d = B.TransitionDesc(N, H, H, cin, cout, k, stride, int(split), eps, mode, frac)
    fb, bb = B.revnet_transition_workspace_bytes(ctx, d)
    ws = torch.empty(max(fb, bb), dtype=torch.uint8, device="cuda")
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    if split:
        in1, in2 = R.to_state(x[:, :cin // 2], frac), R.to_state(x[:, cin // 2:], frac)
    else:
        in1, in2 = dev(B.to_nhwc(x.astype(np.float32))), None
    tW, tg, tb = dev(B.w_to_abi(W)), dev(gamma), dev(beta)
    o1 = torch.empty((N, Ho, Ho, cout // 2), dtype=torch.int32 if frac else torch.float32, device="cuda"); o2 = torch.empty_like(o1)
    B.revnet_transition_fwd(ctx, d, in1, in2, tW, tg, tb, o1, o2, ws)
    y = np.concatenate([R.from_state(o1, frac), R.from_state(o2, frac)], axis=1)
    dyf = dy.astype(np.float32)
    d1, d2 = dev(B.to_nhwc(dyf[:, :cout // 2])), dev(B.to_nhwc(dyf[:, cout // 2:]))
    if split:
        di1 = torch.empty((N, H, H, cin // 2), dtype=torch.float32, device="cuda"); di2 = torch.empty_like(di1)
    else:
        di1, di2 = torch.empty((N, H, H, cin), dtype=torch.float32, device="cuda"), None
    gW, gg, gb = torch.empty_like(tW), torch.empty_like(tg), torch.empty_like(tb)
    B.revnet_transition_bwd(ctx, d, in1, in2, d1, d2, tW, tg, tb, di1, di2, gW, gg, gb, ws)
    torch.cuda.synchronize()
    dx = B.to_nchw(di1.cpu().numpy()) if not split else np.concatenate([B.to_nchw(di1.cpu().numpy()), B.to_nchw(di2.cpu().numpy())], axis=1)
    return dict(y=y, dx=dx, dW=B.w_from_abi(gW.cpu().numpy()), dgamma=gg.cpu().numpy(), dbeta=gb.cpu().numpy())


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("kind,maxpool", [("basic", False), ("bottleneck", False), ("bottleneck", True)])
def test_tiny_stack_parity(ctx, mode, kind, maxpool):
    run_stack_case(ctx, hp.tiny_stack(kind, maxpool, N=6), mode)
    ORACLE_RUNS.clear()


def sample_units(cfg, middle=True):
    """First, (middle) and last unit of every stage."""
    return tuple(sorted({(si, u) for si, s in enumerate(cfg.stages) for u in ((0, s.units // 2, s.units - 1) if middle else (0, s.units - 1))}))


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("name", ["revnet38", "revnet110", "revnet164"])
def test_full_config_parity(ctx, name, mode):
    """BASELINE configs 2, 3 and 4 at full size (batch 128): forward at the stated tolerance; sampled units and
    every transition inside the network at the stated tolerance; end-to-end gradients of the last stage and the
    classifier at the stated tolerance, those in front of it by the floor rule."""
    cfg = syn.stack_config(name)
    keys = sample_units(cfg, middle=(name != "revnet164"))      # (the bottleneck network's oracle runs take minutes: two units per stage)
    frac = R.DEFAULT_FRAC_BITS[mode]
    levels = [2.0 ** -frac] if frac else [1e-6]       # the larger of the rounding differences that exist (one grid step)
    try:
        run_blocks_in_network(ctx, cfg, mode, keys)
        run_stack_case(ctx, cfg, mode, jitter=False, plain_forward=(name == "revnet38" and mode == 1),
                       floor_levels=levels, keep_blocks=keys, keep_transitions=True, logits_floor=(mode == 0 and name == "revnet164"),
                       floor_draws=1)      # millions of elements per layer: one draw already averages over many decisions
    finally:
        ORACLE_RUNS.clear()


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("kind,N,H,c,w", [("basic", 128, 32, 16, 0), ("basic", 128, 16, 32, 0), ("basic", 128, 8, 56, 0),
                                         ("basic", 128, 8, 64, 0), ("bottleneck", 128, 16, 256, 64)])
def test_block_parity_at_benchmark_shapes(ctx, mode, kind, N, H, c, w):
    """One reversible block at the full per-stage shapes of the CIFAR-sized configs (batch 128)."""
    run_block_case(ctx, syn.BlockCfg(N, H, H, c, w, kind, seed=300 + c), mode, jitter=True, inplace=True)


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("name,N,units", [("revnet110", 16, 9), ("revnet164", 8, 2)])
def test_deeper_configs_reduced_batch(ctx, name, N, units, mode):
    """Configs 3 and 4 at their widths with a batch / depth the oracle finishes in seconds."""
    cfg = syn.shrink(syn.stack_config(name), N=N, units=units)
    try:
        run_stack_case(ctx, cfg, mode, jitter=False)
    finally:
        ORACLE_RUNS.clear()


def test_revnet104_shape_reduced(ctx):
    """Config 5's layer kinds (7x7/2 stem, max-pool, entry transition, 4 bottleneck stages) at
    reduced widths and image size."""
    st = tuple(syn.StageCfg(1, 4 * w, w, "bottleneck", 3, 2 if i else 1) for i, w in enumerate((8, 16, 32, 52)))
    cfg = syn.StackCfg("revnet104_small", 4, 64, 20, 7, 2, 16, True, st, seed=4, weight_decay=1e-4)
    try:
        run_stack_case(ctx, cfg, 0, jitter=True, logits_floor=True)      # batch 4: BN over 16 samples in the last stage
        run_stack_case(ctx, cfg, 1, jitter=True)
    finally:
        ORACLE_RUNS.clear()


def test_activation_memory_flat_in_depth_on_device(ctx):
    base = syn.shrink(syn.stack_config("revnet110"), N=8)
    seen = set()
    for units in (1, 3, 9):
        cfg = syn.shrink(base, units=units)
        r = R.StackRunner(ctx, cfg, 0)
        inp = syn.make_stack_inputs(cfg)
        r.load(inp["images"], inp["labels"], inp["params"])
        st = r.step()
        torch.cuda.synchronize()
        seen.add((st.stored_activation_bytes, r.plan.activation_bytes))
        assert np.isfinite(r.results()["loss"])
    assert len(seen) == 1, seen


def test_graph_replay_matches_eager(ctx):
    """The step replayed from its CUDA graph gives the same bits as the step enqueued kernel by kernel."""
    cfg = syn.shrink(syn.stack_config("revnet38"), N=16)
    inp = syn.make_stack_inputs(cfg)
    out = []
    for graph in (False, True):
        r = R.StackRunner(ctx, cfg, 0, use_cuda_graph=graph)
        r.load(inp["images"], inp["labels"], inp["params"])
        for _ in range(3):
            st = r.step()
        res = r.results()
        out.append((res, st))
    (a, sa), (b, sb) = out
    assert a["loss"] == b["loss"] and np.array_equal(a["pred"], b["pred"])
    for k in a["params"]:
        assert np.array_equal(a["params"][k], b["params"][k]), k
        assert np.array_equal(a["grads"][k], b["grads"][k]), k
    assert sa.kernel_launches == sb.kernel_launches and sa.flops_bwd == sb.flops_bwd


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("N,H,cin,cout,k,stride,split", [
    (16, 16, 32, 64, 3, 2, True),     # CIFAR-sized down-sampling transition on a coupling state (tensor-core path)
    (128, 32, 32, 64, 3, 2, True),    # config 2, first transition at full size
    (8, 16, 64, 112, 3, 2, True),     # 112 output channels (56 per half)
    (16, 16, 32, 256, 3, 1, False),   # entry transition from a plain stem output
    (5, 6, 8, 16, 3, 2, True),        # ragged: falls back to the fp32 kernels
    (16, 8, 64, 128, 1, 2, True),     # 1x1 stride 2
    (4, 16, 128, 256, 3, 2, True),    # 128 x 256 tiles in the forward (contraction 1152, 256 output channels)
    (4, 8, 256, 512, 3, 2, True),     # ... and in the parity-class launches of the data gradient (1, 2, 2, 4 taps)
    (4, 14, 64, 128, 3, 2, True),     # 14x14 -> 7x7: tiles of two whole images, class launches on a 7x7 grid
    (2, 28, 128, 256, 3, 1, False),   # 28-wide rows: tiles of 112 pixels, wide tiles with statistics in the epilogue
    (8, 16, 256, 256, 3, 2, True),    # weight gradient of 590 k elements split over four pixel tiles: the tiled sum of the partials
])
def test_stored_transition_layer(ctx, mode, N, H, cin, cout, k, stride, split):
    """BN-ReLU-conv with stride: forward and backward of one stored layer against the oracle."""
    run_transition_case(ctx, mode, N, H, cin, cout, k, stride, split)


def run_transition_case(ctx, mode, N, H, cin, cout, k, stride, split):
    frac = R.DEFAULT_FRAC_BITS[mode]
    rng = np.random.default_rng(1000 + cin + cout + H)
    x = rng.standard_normal((N, cin, H, H)).astype(np.float32)
    Ho = H // stride
    dy = rng.standard_normal((N, cout, Ho, Ho)).astype(np.float32)
    W = (rng.standard_normal((cout, cin, k, k)) * np.sqrt(2.0 / (cin * k * k))).astype(np.float32)
    gamma = (1 + 0.1 * rng.standard_normal(cin)).astype(np.float32); beta = (0.1 * rng.standard_normal(cin)).astype(np.float32)
    num = {}
    if mode == 0: num["bf16_operands"] = True
    if frac: num["frac_bits"] = frac
    num = num or None
    x64 = x.astype(np.float64)
    if split and frac:
        x64 = np.rint(x64 * (1 << frac)) / (1 << frac)
    layer = [dict(name="T", gamma=gamma, beta=beta, W=W, stride=stride)]
    oy, cache = orc.fn_fwd(x64, layer, 1e-5, num)
    oy = orc.quantize_state(oy, num)
    og = {}
    odx = orc.fn_bwd(dy.astype(np.float64), cache, og, num)
    got = transition_through_abi(ctx, x64, dy.astype(np.float64), W, gamma, beta, stride, split, mode, frac, 1e-5)
    case = f"transition N{N} {H}x{H} {cin}->{cout} k{k} s{stride} split{int(split)} mode{mode}"
    par.check(case + " fwd", dict(y=got["y"]), dict(y=oy), 1e-4 if mode else 2e-3)
    tol = 1e-4 if mode else 1e-2          # one layer deep: far inside the stated 5e-2
    par.check(case + " bwd", {"dx": got["dx"], "T.W": got["dW"], "T.gamma": got["dgamma"], "T.beta": got["dbeta"]},
              {"dx": odx, "T.W": og["T.W"], "T.gamma": og["T.gamma"], "T.beta": og["T.beta"]}, tol)


@pytest.mark.parametrize("mode", [0, 1])
def test_shallow_stack_with_stride2_transitions(ctx, mode):
    """Three stages of one unit each with two stride-2 stored transitions."""
    st = (syn.StageCfg(1, 8, 0, "basic", 0, 1), syn.StageCfg(1, 16, 0, "basic", 3, 2), syn.StageCfg(1, 32, 0, "basic", 3, 2))
    cfg = syn.StackCfg("shallow_s2", 16, 16, 7, 3, 1, 16, False, st, seed=31)
    run_stack_case(ctx, cfg, mode)
    ORACLE_RUNS.clear()


def paper_tiny(kind, N=6):
    """A small network shaped like the paper's table: the first unit of stages 2.. carries the down-sampling."""
    if kind == "basic":
        st = (syn.StageCfg(2, 8, 0, "basic", 0, 1), syn.StageCfg(2, 16, 0, "basic", 0, 1, down=True), syn.StageCfg(1, 24, 0, "basic", 0, 1, down=True))
        stem_c = 16
    else:
        st = (syn.StageCfg(1, 16, 8, "bottleneck", 3, 1), syn.StageCfg(2, 32, 8, "bottleneck", 0, 1, down=True), syn.StageCfg(2, 64, 16, "bottleneck", 0, 1, down=True))
        stem_c = 8
    return syn.StackCfg(f"paper_tiny_{kind}", N, 16, 5, 3, 1, stem_c, False, st, seed=17)


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("kind", ["basic", "bottleneck"])
def test_paper_shaped_tiny_stack_parity(ctx, kind, mode):
    """Down-sampling inside the first unit of a stage (Table "Architectural details"): stored coupling unit with a
    stride-2 layer in F and average-pool shortcuts, followed by reversible units."""
    try:
        run_stack_case(ctx, paper_tiny(kind), mode)
    finally:
        ORACLE_RUNS.clear()


@pytest.mark.parametrize("mode", [1, 0])
def test_paper_revnet38_reduced_batch(ctx, mode):
    """The table's RevNet-38 (units 3-3-3, widths 32/64/112, no separate transitions) at batch 16."""
    cfg = syn.shrink(syn.stack_config("paper_revnet38"), N=16)
    try:
        run_stack_case(ctx, cfg, mode, jitter=False)
    finally:
        ORACLE_RUNS.clear()
