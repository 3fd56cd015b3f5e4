"""The stored-activation train step (store_activations = 1): ordinary backprop on what the forward
pass kept, the baseline the reversible step is traded against (Section 3.2).

Both steps compute the same gradients (Section 3: reversing the units changes where the activations
come from, not what is differentiated), so the stored step is checked against the reversible one
run on the same inputs -- bit for bit in the bf16 mode with its fixed-point state, where the
reversal reproduces every tensor of the forward pass exactly -- and, in strict mode, against the
oracle's stored-activation flavour.  Its storage must grow with the number of units while the
reversible step's does not.
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


def both_steps(ctx, cfg, mode, graph):
    inp = syn.make_stack_inputs(cfg, affine_jitter=True)
    out = []
    for stored in (False, True):
        r = R.StackRunner(ctx, cfg, mode, use_cuda_graph=graph, store_activations=stored)
        r.load(inp["images"], inp["labels"], inp["params"])
        st = r.step()
        if graph:                       # second call replays the captured graph from the same state
            r.load(inp["images"], inp["labels"], inp["params"])
            st = r.step()
        out.append((r.results(), st))
        B.revnet_check_device(ctx)
    return inp, out


@pytest.mark.parametrize("graph", [False, True])
@pytest.mark.parametrize("kind,maxpool", [("basic", False), ("bottleneck", False), ("bottleneck", True)])
def test_stored_step_equals_reversible_step_bitwise_in_bf16_mode(ctx, kind, maxpool, graph):
    cfg = hp.tiny_stack(kind, maxpool, N=6, units=3)
    _, ((rev, srev), (sto, ssto)) = both_steps(ctx, cfg, 0, graph)
    assert np.array_equal(rev["logits"], sto["logits"]) and rev["loss"] == sto["loss"]
    for k in rev["grads"]:
        assert np.array_equal(rev["grads"][k], sto["grads"][k]), k
        assert np.array_equal(rev["params"][k], sto["params"][k]), k
    # the stored step skips the recomputation: three conv passes per reversible layer instead of four
    assert ssto.flops_fwd == srev.flops_fwd and ssto.flops_bwd < srev.flops_bwd
    assert ssto.stored_activation_bytes > srev.stored_activation_bytes


@pytest.mark.parametrize("kind,maxpool", [("basic", False), ("bottleneck", True)])
def test_stored_step_strict_mode_against_oracle_and_reversible(ctx, kind, maxpool):
    cfg = hp.tiny_stack(kind, maxpool, N=6, units=2)
    inp, ((rev, _), (sto, _)) = both_steps(ctx, cfg, 1, False)
    net = hp.oracle_net(cfg, inp["params"])
    o = orc.stack_train_grads(net, inp["images"], inp["labels"], "stored")
    assert hp.rel_l2(sto["logits"], o["logits"]) <= 1e-4
    for k in o["grads"]:
        assert hp.rel_l2(sto["grads"][k], o["grads"][k]) <= 1e-4, k
        assert hp.rel_l2(sto["grads"][k], rev["grads"][k]) <= 1e-4, k


def test_stored_step_at_benchmark_width_and_storage_growth(ctx):
    """RevNet-38 widths at batch 16: gradients equal the reversible step's; kept bytes grow linearly in depth."""
    base = syn.shrink(syn.stack_config("revnet38"), N=16)
    _, ((rev, srev), (sto, ssto)) = both_steps(ctx, base, 0, True)
    for k in rev["grads"]:
        assert np.array_equal(rev["grads"][k], sto["grads"][k]), k
    kept = {}
    for units in (1, 2, 4):
        cfg = syn.shrink(base, units=units)
        sizes = []
        for stored in (False, True):
            r = R.StackRunner(ctx, cfg, 0, store_activations=stored)
            inp = syn.make_stack_inputs(cfg)
            r.load(inp["images"], inp["labels"], inp["params"])
            sizes.append(int(r.step().stored_activation_bytes))
            torch.cuda.synchronize()
        kept[units] = sizes
    assert kept[1][0] == kept[2][0] == kept[4][0]                       # reversible: flat in depth
    assert kept[4][1] - kept[2][1] == 2 * (kept[2][1] - kept[1][1]) > 0   # stored: the same amount per unit


@pytest.mark.parametrize("name", ["revnet110", "revnet164"])
def test_stored_step_equals_reversible_step_at_full_size(ctx, name):
    """The deep configurations at full batch, graph replay (the benchmark's launch configuration): both steps end
    with the same bits in every gradient and updated weight, the stored one with less backward work."""
    cfg = syn.stack_config(name)
    inp = syn.make_stack_inputs(cfg)
    flat = []
    stats = []
    for stored in (False, True):
        r = R.StackRunner(ctx, cfg, 0, store_activations=stored)
        r.load(inp["images"], inp["labels"], inp["params"])
        r.step(want_logits=False)                      # captures the graph
        r.load(inp["images"], inp["labels"], inp["params"])
        stats.append(r.step(want_logits=False))        # replays it from the same state
        torch.cuda.synchronize()
        flat.append((r.grads.clone(), r.params.clone(), float(r.loss.item())))
        B.revnet_check_device(ctx)
        del r
        torch.cuda.empty_cache()
    assert torch.equal(flat[0][0], flat[1][0]) and torch.equal(flat[0][1], flat[1][1]) and flat[0][2] == flat[1][2]
    assert np.isfinite(flat[0][2])
    assert stats[1].flops_bwd < stats[0].flops_bwd and stats[1].stored_activation_bytes > 5 * stats[0].stored_activation_bytes


def test_profiled_step_gives_the_same_result(ctx):
    """Per-kernel profiling runs the step on one stream, kernel by kernel (no side streams, no graph).  The forward
    pass is the same launches, hence the same bits; the weight gradients of a function are then one launch per layer
    instead of one per function, which splits their pixel sums differently: equal up to float32 summation order."""
    cfg = syn.shrink(syn.stack_config("revnet38"), N=16)
    inp = syn.make_stack_inputs(cfg, affine_jitter=True)
    res = []
    for profiled in (False, True):
        r = R.StackRunner(ctx, cfg, 0)
        r.load(inp["images"], inp["labels"], inp["params"])
        if profiled:
            B.revnet_profile_enable(ctx, 2)
        r.step()
        torch.cuda.synchronize()
        if profiled:
            prof = B.revnet_profile_summary(ctx)
            B.revnet_profile_enable(ctx, 0)
            assert any(k.startswith("conv_fprop_fused|") for k in prof) and all(v["ms"] >= 0 for v in prof.values())
        res.append((r.grads.clone(), r.params.clone(), r.logits.clone()))
        B.revnet_check_device(ctx)
    assert torch.equal(res[0][2], res[1][2])
    for a, b in zip(res[0][:2], res[1][:2]):
        assert float((a - b).norm() / b.norm()) <= 1e-5
