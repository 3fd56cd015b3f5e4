"""The train step at the FULL sizes of the deep configurations, in the launch configuration bench.py
times (bf16 mode, fixed-point state, CUDA-graph replay where the step allows it).

The oracle cannot run these sizes in reasonable time (BN couples the whole batch, so the batch
cannot be sub-sampled), hence:
  - sampled outputs the oracle computes one by one: the stem convolution (what the first stored
    tensor holds after the step) at random pixels, from the oracle's direct-loop convolution;
  - properties that hold at any size: every stage reconstructs its input bit for bit (Section 3.1,
    fixed-point state), the loss equals the softmax cross-entropy of the returned logits and the
    predictions their arg-max (oracle's softmax_ce), the SGD update is the closed form of
    Appendix 6.1 applied to the returned gradients, stored activation bytes do not depend on the
    number of units per stage (Section 3.2), and a second run from the same state gives the same bits.
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


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    B.revnet_check_device(c)
    c.close()


def stem_samples(cfg, inp, n_samples, rng):
    """Oracle values of the stem convolution at random output pixels: (n, i, j) -> [stem_cout]."""
    Hs = (cfg.img + 2 * cfg.stem_pad - cfg.stem_k) // cfg.stem_stride + 1
    W = inp["params"]["stem.W"].astype(np.float64)
    k, p, s = cfg.stem_k, cfg.stem_pad, cfg.stem_stride
    out = []
    for _ in range(n_samples):
        n, i, j = int(rng.integers(cfg.N)), int(rng.integers(Hs)), int(rng.integers(Hs))
        patch = np.zeros((1, cfg.in_ch, k, k))
        for kh in range(k):
            for kw in range(k):
                y, x = i * s + kh - p, j * s + kw - p
                if 0 <= y < cfg.img and 0 <= x < cfg.img:
                    patch[0, :, kh, kw] = inp["images"][n, :, y, x]
        out.append(((n, i, j), orc.conv_fwd(patch, W, stride=1, pad=0)[0, :, 0, 0]))
    return Hs, out


def full_size_case(ctx, cfg, n_samples=64):
    inp = syn.make_stack_inputs(cfg)
    specs = syn.param_specs(cfg)
    flat0 = B.pack_params(specs, inp["params"])

    # ---- run 1: reconstruction check on (no graph), logits returned
    r = R.StackRunner(ctx, cfg, 0, verify_reconstruction=True)
    r.load(inp["images"], inp["labels"], inp["params"])
    st = r.step()
    torch.cuda.synchronize()
    for si in range(len(cfg.stages)):
        assert st.recon_max_abs[si] == 0.0, (si, st.recon_max_abs[si])      # bit-exact inversion at every stage
    logits = r.logits.cpu().numpy().astype(np.float64)
    assert np.isfinite(logits).all()
    loss, pred = float(r.loss.item()), r.pred.cpu().numpy()
    # loss / predictions from the returned logits (oracle's softmax cross-entropy)
    ref_loss, _ = orc.softmax_ce(logits, inp["labels"])
    assert abs(loss - ref_loss) <= 1e-4 * max(1.0, abs(ref_loss))
    assert np.array_equal(pred, logits.argmax(axis=1).astype(np.int32))

    # ---- SGD closed form on the returned gradients (v0 = 0): v = g + wd*w (conv / FC weights), w' = w - lr*v
    g = r.grads.cpu().numpy().astype(np.float64)
    v = r.momentum.cpu().numpy().astype(np.float64)
    w1 = r.params.cpu().numpy().astype(np.float64)
    decay = np.zeros(flat0.size, bool)
    o = 0
    for name, shape, role in specs:
        n = int(np.prod(shape))
        if role in ("convw", "fcw"):
            decay[o:o + n] = True
        o += n
    v_ref = g + np.where(decay, cfg.weight_decay * flat0.astype(np.float64), 0.0)
    assert np.isfinite(g).all()
    assert np.abs(v - v_ref).max() <= 1e-6 * max(1.0, np.abs(v_ref).max())
    assert np.abs(w1 - (flat0 - cfg.lr * v_ref)).max() <= 1e-6 * max(1.0, np.abs(flat0).max())
    # every parameter tensor received a gradient
    o = 0
    for name, shape, role in specs:
        n = int(np.prod(shape))
        assert np.abs(g[o:o + n]).max() > 0, name
        o += n

    # ---- sampled stem outputs: the first stored tensor is the stem output (stage 0's x1 in the state
    # format when the stem feeds stage 0 directly)
    rng = np.random.default_rng(7)
    Hs, samples = stem_samples(cfg, inp, n_samples, rng)
    direct = (not cfg.maxpool) and cfg.stages[0].trans_k == 0
    cw = cfg.stages[0].c if direct else cfg.stem_cout
    n_el = cfg.N * Hs * Hs * cw
    first = r.act[: n_el * 4].view(torch.int32 if direct else torch.float32).reshape(cfg.N, Hs, Hs, cw).cpu().numpy()
    for (n, i, j), ref in samples:
        got = first[n, i, j].astype(np.float64)
        if direct:
            got = got / (1 << r.frac)
            assert np.abs(got - ref[:cw]).max() <= 2.0 ** -(r.frac + 1) + 1e-5 * max(1.0, np.abs(ref).max())
        else:
            assert np.abs(got - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max())

    # ---- run 2: the benchmark's configuration (graph replay), same start: same bits
    r2 = R.StackRunner(ctx, cfg, 0, use_cuda_graph=True)
    r2.load(inp["images"], inp["labels"], inp["params"])
    st2 = r2.step()
    torch.cuda.synchronize()
    assert float(r2.loss.item()) == loss
    assert torch.equal(r2.grads, r.grads) and torch.equal(r2.params, r.params)
    assert st2.stored_activation_bytes == st.stored_activation_bytes
    # storage independent of depth: the plan of the same network with other unit counts stores the same bytes
    for units in (1, 18):
        pl = B.revnet_stack_plan(ctx, B.stack_desc(syn.shrink(cfg, units=units), 0, False, r.frac, False))
        assert pl.activation_bytes == r2.plan.activation_bytes
        pl.close()
    return st


def test_revnet110_full_size(ctx):
    full_size_case(ctx, syn.stack_config("revnet110"))


def test_revnet164_full_size(ctx):
    full_size_case(ctx, syn.stack_config("revnet164"))


def test_revnet104_full_size(ctx):
    """Config 5: batch 64 of 224x224, 491 M parameters."""
    full_size_case(ctx, syn.stack_config("revnet104"), n_samples=16)
