"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Tolerances (relative L2 per tensor unless stated):
  strict fp32 mode : 1e-4 everywhere
  bf16 mode        : block outputs / logits 2e-2, gradients 5e-2
  reconstruction   : recovered x1, x2 within 1e-3 max-abs of the inputs that produced y1, y2
  integers (arg-max predictions) : exact
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


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    c.close()


def run_block_case(ctx, b, mode, jitter, inplace):
    inp = syn.make_block_inputs(b, affine_jitter=jitter)
    F, G = hp.oracle_block(b, inp["params"])
    x1, x2, dy1, dy2 = (inp[k].astype(np.float64) for k in ("x1", "x2", "dy1", "dy2"))
    oy1, oy2 = orc.block_fwd(x1, x2, F, G, b.eps)
    og = {}
    ox1, ox2, odx1, odx2 = orc.block_bwd_reconstruct(oy1, oy2, dy1, dy2, F, G, b.eps, og)
    r = R.BlockRunner(ctx, b, mode)
    r.load(inp["params"])
    y1, y2 = r.forward(inp["x1"], inp["x2"], inplace=inplace)
    t = TOL[mode]
    assert hp.rel_l2(y1, oy1) <= t["out"] and hp.rel_l2(y2, oy2) <= t["out"]
    # backward from the GPU's own outputs: reconstruction must return the inputs that produced them
    rx1, rx2, dx1, dx2, grads = r.backward(y1, y2, inp["dy1"], inp["dy2"], inplace=inplace)
    assert np.abs(rx1 - inp["x1"]).max() <= RECON and np.abs(rx2 - inp["x2"]).max() <= RECON
    assert hp.rel_l2(dx1, odx1) <= t["grad"] and hp.rel_l2(dx2, odx2) <= t["grad"]
    assert set(grads) == set(og)
    for k in og:
        assert hp.rel_l2(grads[k], og[k]) <= t["grad"], (k, hp.rel_l2(grads[k], og[k]))
    return dict(recon=max(np.abs(rx1 - inp["x1"]).max(), np.abs(rx2 - inp["x2"]).max()))


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
    assert worst <= RECON, worst


def run_stack_case(ctx, cfg, mode, jitter=True):
    inp = syn.make_stack_inputs(cfg, affine_jitter=jitter)
    net = hp.oracle_net(cfg, inp["params"])
    o = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct")
    zero_v = {k: np.zeros_like(v, dtype=np.float64) for k, v in inp["params"].items()}
    op, ov = orc.sgd_step(inp["params"], o["grads"], zero_v, cfg.lr, cfg.momentum, cfg.weight_decay, hp.decayed_names(cfg))
    r = R.StackRunner(ctx, cfg, mode, verify_reconstruction=True)
    r.load(inp["images"], inp["labels"], inp["params"])
    st = r.step()
    g = r.results()
    t = TOL[mode]
    assert hp.rel_l2(g["logits"], o["logits"]) <= t["out"], hp.rel_l2(g["logits"], o["logits"])
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
    worst = {}
    for k in o["grads"]:
        e = hp.rel_l2(g["grads"][k], o["grads"][k])
        worst[k] = e
        assert e <= t["grad"], (k, e)
    for k in op:
        assert hp.rel_l2(g["params"][k], op[k]) <= t["grad"], k
        assert hp.rel_l2(g["momentum"][k], ov[k]) <= t["grad"], k
    for si in range(len(cfg.stages)):
        assert st.recon_max_abs[si] <= RECON, (si, st.recon_max_abs[si])
    assert st.stored_activation_bytes == o["stored_bytes"]
    return st, max(worst.values())


@pytest.mark.parametrize("mode", [1, 0])
@pytest.mark.parametrize("kind,maxpool", [("basic", False), ("bottleneck", False), ("bottleneck", True)])
def test_tiny_stack_parity(ctx, mode, kind, maxpool):
    run_stack_case(ctx, hp.tiny_stack(kind, maxpool, N=6), mode)


@pytest.mark.parametrize("mode", [1, 0])
def test_revnet38_full_config_parity(ctx, mode):
    """BASELINE config 2 at full size: batch 128, 3 stages of 3 basic units at 32/64/112 channels."""
    run_stack_case(ctx, syn.stack_config("revnet38"), mode, jitter=False)


@pytest.mark.parametrize("name,N,units", [("revnet110", 16, 9), ("revnet164", 8, 2)])
def test_deeper_configs_reduced_batch(ctx, name, N, units):
    """Configs 3 and 4 at their widths with a batch / depth the oracle finishes in seconds."""
    run_stack_case(ctx, syn.shrink(syn.stack_config(name), N=N, units=units), 0, jitter=False)


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
