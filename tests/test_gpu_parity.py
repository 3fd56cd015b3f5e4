"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Tolerances (relative L2 per tensor unless stated):
  strict fp32 mode : 1e-4 everywhere
  bf16 mode        : block outputs / logits 2e-2, gradients 5e-2
  reconstruction   : recovered x1, x2 within 1e-3 max-abs of the inputs that produced y1, y2;
                     on the fixed-point coupling state (the bf16 mode's default) they are bit-exact
  integers (arg-max predictions) : exact

Conditioning.  The gradient of a BN-ReLU network is a discontinuous function of its activations:
an element whose pre-activation changes sign moves a whole term in or out of every sum behind it.
Rounding differences between any two implementations flip a few such elements per layer once a
layer has millions of them, and bf16 operand rounding feeds the flips back into later layers.  So
for large or deep cases the oracle's OWN gradients move by more than the stated tolerance when
its input is perturbed by 1e-6 (relative).  Where a case misses the stated tolerance, the test
measures that self-sensitivity ("floor") with further oracle runs (input perturbed by 1e-6 and, on
a fixed-point state, by one grid step, the two sizes of rounding difference that exist between the
kernel and the oracle) and accepts an error up to FLOOR_FACTOR x floor, capped at MAX_BOUND; cases
that nothing tips over (floor ~ 0) are therefore held to the stated numbers.
"""
import numpy as np
import pytest
import torch

from oracle import revnet as orc
from paper_1707_04585_b200 import binding as B
from paper_1707_04585_b200 import runner as R
from paper_1707_04585_b200 import synthetic as syn
from tests import helpers as hp

pytestmark = pytest.mark.gpu

TOL = {1: dict(out=1e-4, grad=1e-4), 0: dict(out=2e-2, grad=5e-2)}
RECON = 1e-3
FLOOR_FACTOR = 3.0
MAX_BOUND = 1.5          # beyond this a gradient is anti-aligned with the oracle's


def check_grads(got, ref, tol, floor_fn, levels, what):
    """Every tensor within `tol`; failing that, within FLOOR_FACTOR x the oracle's self-sensitivity."""
    errs = {k: hp.rel_l2(got[k], ref[k]) for k in ref}
    if max(errs.values()) <= tol:
        return max(errs.values()), 0.0
    floor = 0.0
    for level in levels:
        floor_ref = floor_fn(level)
        floor = max(floor, max(hp.rel_l2(floor_ref[k], ref[k]) for k in ref))
    bound = min(MAX_BOUND, max(tol, FLOOR_FACTOR * floor))
    bad = {k: e for k, e in errs.items() if e > bound}
    assert not bad, f"{what}: errors {bad} exceed max(tol {tol}, {FLOOR_FACTOR} x floor {floor:.3e})"
    return max(errs.values()), floor


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


def run_block_case(ctx, b, mode, jitter, inplace):
    inp = syn.make_block_inputs(b, affine_jitter=jitter)
    F, G = hp.oracle_block(b, inp["params"])
    r = R.BlockRunner(ctx, b, mode)
    r.load(inp["params"])
    num = oracle_numerics(r)
    x1, x2, dy1, dy2 = (inp[k].astype(np.float64) for k in ("x1", "x2", "dy1", "dy2"))
    grid = float(1 << r.frac) if r.frac else None
    if grid:
        x1, x2 = np.rint(x1 * grid) / grid, np.rint(x2 * grid) / grid

    def oracle(x1_, x2_):
        y1_, y2_ = orc.block_fwd(x1_, x2_, F, G, b.eps, num=num)
        g_ = {}
        _, _, dx1_, dx2_ = orc.block_bwd_reconstruct(y1_, y2_, dy1, dy2, F, G, b.eps, g_, num=num)
        g_["dx1"], g_["dx2"] = dx1_, dx2_
        return y1_, y2_, g_

    py1, py2 = orc.block_fwd(x1, x2, F, G, b.eps)                    # the plain float64 definition
    oy1, oy2, og = oracle(x1, x2)
    y1, y2 = r.forward(inp["x1"], inp["x2"], inplace=inplace)
    t = TOL[mode]
    assert hp.rel_l2(y1, py1) <= t["out"] and hp.rel_l2(y2, py2) <= t["out"]
    assert hp.rel_l2(y1, oy1) <= t["out"] and hp.rel_l2(y2, oy2) <= t["out"]
    # backward from the GPU's own outputs: reconstruction must return the inputs that produced them
    rx1, rx2, dx1, dx2, grads = r.backward(y1, y2, inp["dy1"], inp["dy2"], inplace=inplace)
    assert np.abs(rx1 - x1).max() <= RECON and np.abs(rx2 - x2).max() <= RECON
    if grid:        # fixed-point state: the inputs as the kernel saw them come back bit for bit
        assert np.array_equal(rx1, x1) and np.array_equal(rx2, x2)
    grads["dx1"], grads["dx2"] = dx1, dx2
    assert set(grads) == set(og)

    def floor_fn(level):
        rng = np.random.default_rng(99)
        p1 = x1 * (1 + level * rng.uniform(-1, 1, x1.shape)); p2 = x2 * (1 + level * rng.uniform(-1, 1, x2.shape))
        if grid:
            p1, p2 = np.rint(p1 * grid) / grid, np.rint(p2 * grid) / grid
        return oracle(p1, p2)[2]
    return check_grads(grads, og, t["grad"], floor_fn, perturb_levels(r), f"block {b}")


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


def run_stack_case(ctx, cfg, mode, jitter=True, plain_forward=False):
    inp = syn.make_stack_inputs(cfg, affine_jitter=jitter)
    net = hp.oracle_net(cfg, inp["params"])
    r = R.StackRunner(ctx, cfg, mode, verify_reconstruction=True)
    o = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct", num=oracle_numerics(r))
    zero_v = {k: np.zeros_like(v, dtype=np.float64) for k, v in inp["params"].items()}
    op, ov = orc.sgd_step(inp["params"], o["grads"], zero_v, cfg.lr, cfg.momentum, cfg.weight_decay, hp.decayed_names(cfg))
    r.load(inp["images"], inp["labels"], inp["params"])
    st = r.step()
    g = r.results()
    t = dict(TOL[mode])
    floor_runs = {}

    def floor_run(level):
        if level not in floor_runs:
            rng = np.random.default_rng(98)
            pim = inp["images"].astype(np.float64) * (1 + level * rng.uniform(-1, 1, inp["images"].shape))
            floor_runs[level] = orc.stack_train_grads(net, pim, inp["labels"], "reconstruct", num=oracle_numerics(r))
        return floor_runs[level]

    # logits: the stated tolerance, unless one rounding decision tipping over already moves the oracle's
    # own logits further than that (tiny batches: BN over a few dozen samples), see the module docstring
    check_grads(dict(logits=g["logits"]), dict(logits=o["logits"]), t["out"], lambda lv: dict(logits=floor_run(lv)["logits"]),
                perturb_levels(r), cfg.name + " logits")
    if plain_forward:       # forward quantities also against the unrounded float64 definition
        plain = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct")
        assert hp.rel_l2(g["logits"], plain["logits"]) <= t["out"]
    assert abs(g["loss"] - o["loss"]) <= t["out"] * max(1.0, abs(o["loss"]))
    # arg-max: the kernel must agree exactly with the arg-max of its own logits, and with the oracle
    # wherever the oracle's top-2 margin exceeds the logit tolerance
    assert np.array_equal(g["pred"], g["logits"].argmax(axis=1).astype(np.int32))
    srt = np.sort(o["logits"], axis=1)
    margin = srt[:, -1] - srt[:, -2]
    clear = margin > 2 * t["out"] * np.abs(o["logits"]).max()
    assert np.array_equal(g["pred"][clear], o["pred"][clear])
    if mode == 1:
        assert np.array_equal(g["pred"], o["pred"])
    worst, floor = check_grads(g["grads"], o["grads"], t["grad"], lambda lv: floor_run(lv)["grads"], perturb_levels(r), cfg.name)
    bound = min(MAX_BOUND, max(t["grad"], FLOOR_FACTOR * floor))
    for k in op:
        # momentum = gradient + weight decay; updated weights move by lr * momentum
        assert hp.rel_l2(g["momentum"][k], ov[k]) <= bound, k
        assert hp.rel_l2(g["params"][k], op[k]) <= bound, k
    for si in range(len(cfg.stages)):
        assert st.recon_max_abs[si] <= RECON, (si, st.recon_max_abs[si])
        if r.frac:
            assert st.recon_max_abs[si] == 0.0, (si, st.recon_max_abs[si])   # fixed-point state: exact
    assert st.stored_activation_bytes == o["stored_bytes"]
    return st, worst, floor


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("kind,maxpool", [("basic", False), ("bottleneck", False), ("bottleneck", True)])
def test_tiny_stack_parity(ctx, mode, kind, maxpool):
    run_stack_case(ctx, hp.tiny_stack(kind, maxpool, N=6), mode)


@pytest.mark.parametrize("mode", [1, 0])
def test_revnet38_full_config_parity(ctx, mode):
    """BASELINE config 2 at full size: batch 128, 3 stages of 3 basic units at 32/64/112 channels."""
    run_stack_case(ctx, syn.stack_config("revnet38"), mode, jitter=False, plain_forward=True)


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
    run_stack_case(ctx, syn.shrink(syn.stack_config(name), N=N, units=units), mode, jitter=False)


def test_revnet104_shape_reduced(ctx):
    """Config 5's layer kinds (7x7/2 stem, max-pool, entry transition, 4 bottleneck stages) at
    reduced widths and image size."""
    st = tuple(syn.StageCfg(1, 4 * w, w, "bottleneck", 3, 2 if i else 1) for i, w in enumerate((8, 16, 32, 52)))
    cfg = syn.StackCfg("revnet104_small", 4, 64, 20, 7, 2, 16, True, st, seed=4, weight_decay=1e-4)
    run_stack_case(ctx, cfg, 0, jitter=True)
    run_stack_case(ctx, cfg, 1, jitter=True)


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

    d = B.TransitionDesc(N, H, H, cin, cout, k, stride, int(split), 1e-5, mode, frac)
    fb, bb = B.revnet_transition_workspace_bytes(ctx, d)
    ws = torch.empty(max(fb, bb), dtype=torch.uint8, device="cuda")
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    if split:
        in1, in2 = R.to_state(x[:, :cin // 2], frac), R.to_state(x[:, cin // 2:], frac)
    else:
        in1, in2 = dev(B.to_nhwc(x)), None
    tW, tg, tb = dev(B.w_to_abi(W)), dev(gamma), dev(beta)
    o1 = torch.empty((N, Ho, Ho, cout // 2), dtype=torch.int32 if frac else torch.float32, device="cuda"); o2 = torch.empty_like(o1)
    B.revnet_transition_fwd(ctx, d, in1, in2, tW, tg, tb, o1, o2, ws)
    y = np.concatenate([R.from_state(o1, frac), R.from_state(o2, frac)], axis=1)
    t = TOL[mode]
    assert hp.rel_l2(y, oy) <= (1e-4 if mode else 2e-3), hp.rel_l2(y, oy)
    d1, d2 = dev(B.to_nhwc(dy[:, :cout // 2])), dev(B.to_nhwc(dy[:, cout // 2:]))
    if split:
        di1 = torch.empty((N, H, H, cin // 2), dtype=torch.float32, device="cuda"); di2 = torch.empty_like(di1)
    else:
        di1, di2 = torch.empty((N, H, H, cin), dtype=torch.float32, device="cuda"), None
    gW, gg, gb = torch.empty_like(tW), torch.empty_like(tg), torch.empty_like(tb)
    B.revnet_transition_bwd(ctx, d, in1, in2, d1, d2, tW, tg, tb, di1, di2, gW, gg, gb, ws)
    torch.cuda.synchronize()
    dx = B.to_nchw(di1.cpu().numpy()) if not split else np.concatenate([B.to_nchw(di1.cpu().numpy()), B.to_nchw(di2.cpu().numpy())], axis=1)
    tol = 1e-4 if mode else 1e-2          # one layer deep: far inside the stated 5e-2
    assert hp.rel_l2(dx, odx) <= tol, hp.rel_l2(dx, odx)
    assert hp.rel_l2(B.w_from_abi(gW.cpu().numpy()), og["T.W"]) <= tol
    assert hp.rel_l2(gg.cpu().numpy(), og["T.gamma"]) <= tol and hp.rel_l2(gb.cpu().numpy(), og["T.beta"]) <= tol


@pytest.mark.parametrize("mode", [0, 1])
def test_shallow_stack_with_stride2_transitions(ctx, mode):
    """Three stages of one unit each with two stride-2 stored transitions."""
    st = (syn.StageCfg(1, 8, 0, "basic", 0, 1), syn.StageCfg(1, 16, 0, "basic", 3, 2), syn.StageCfg(1, 32, 0, "basic", 3, 2))
    cfg = syn.StackCfg("shallow_s2", 16, 16, 7, 3, 1, 16, False, st, seed=31)
    run_stack_case(ctx, cfg, mode)
