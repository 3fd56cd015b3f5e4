"""Boundary behaviour on the device: pre-packed weights give the same bits as packing per call, a
bounded wait that runs out is reported and leaves the context usable, a label out of range is
reported instead of followed, undersized declared buffers are refused."""
import numpy as np
import pytest
import torch

from oracle import revnet as orc
from paper_1707_04585_b200 import binding as B
from paper_1707_04585_b200 import runner as R
from paper_1707_04585_b200 import synthetic as syn
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kind,N,H,c,w", [("basic", 8, 16, 32, 0), ("bottleneck", 4, 8, 128, 32), ("basic", 2, 8, 40, 0)])
def test_prepacked_weights_give_the_same_bits(kind, N, H, c, w):
    ctx = B.Context(0)
    b = syn.BlockCfg(N, H, H, c, w, kind, seed=9)
    inp = syn.make_block_inputs(b, affine_jitter=True)
    outs = []
    for packed in (False, True):
        r = R.BlockRunner(ctx, b, 0)
        r.load(inp["params"])
        if packed:
            r.pack()
            assert all(l["Wpack_fprop"] and l["Wpack_dgrad"] for l in r.F + r.G)
        y = r.forward(inp["x1"], inp["x2"])
        g = r.backward(y[0], y[1], inp["dy1"], inp["dy2"])
        outs.append((y, g))
    (ya, ga), (yb, gb) = outs
    assert np.array_equal(ya[0], yb[0]) and np.array_equal(ya[1], yb[1])
    for u, v in zip(ga[:4], gb[:4]):
        assert np.array_equal(u, v)
    for k in ga[4]:
        assert np.array_equal(ga[4][k], gb[4][k]), k
    B.revnet_check_device(ctx)
    ctx.close()


def test_pack_buffer_checks():
    ctx = B.Context(0)
    b = syn.BlockCfg(2, 8, 8, 32, 0, "basic", seed=9)
    r = R.BlockRunner(ctx, b, 0)
    r.load(syn.make_block_inputs(b)["params"])
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.RevnetError, match="needed") as e:
        B.revnet_pack_weights(ctx, r.desc, r.F, r.G, small)
    assert e.value.status == -3          # REVNET_E_WORKSPACE_TOO_SMALL
    ctx.close()


def test_bounded_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    """A kernel waits at most 1 ms on a barrier nothing arrives on, gives up, records the status and returns."""
    ctx = B.Context(0)
    B.revnet_selftest_bounded_wait(ctx, 1_000_000)
    with pytest.raises(B.RevnetError) as e:
        B.revnet_check_device(ctx)
    assert e.value.status == -6          # REVNET_E_TIMEOUT
    B.revnet_check_device(ctx)           # cleared: reported once
    # the next regular call works and still matches the oracle
    b = syn.block_config_1()
    inp = syn.make_block_inputs(b)
    F, G = hp.oracle_block(b, inp["params"])
    oy1, oy2 = orc.block_fwd(inp["x1"].astype(np.float64), inp["x2"].astype(np.float64), F, G, b.eps)
    r = R.BlockRunner(ctx, b, 1)
    r.load(inp["params"])
    y1, y2 = r.forward(inp["x1"], inp["x2"])
    assert hp.rel_l2(y1, oy1) <= 1e-4 and hp.rel_l2(y2, oy2) <= 1e-4
    B.revnet_check_device(ctx)
    ctx.close()


def test_label_out_of_range_is_reported_not_followed():
    ctx = B.Context(0)
    cfg = hp.tiny_stack("basic", N=8)
    inp = syn.make_stack_inputs(cfg)
    r = R.StackRunner(ctx, cfg, 1, use_cuda_graph=False)
    labels = inp["labels"].copy()
    labels[3] = cfg.n_classes + 1000000          # far outside: followed, it would read ~4 MB past the logits
    r.load(inp["images"], labels, inp["params"])
    r.step()
    torch.cuda.synchronize()
    assert np.isnan(float(r.loss.item()))
    with pytest.raises(B.RevnetError) as e:
        B.revnet_check_device(ctx)
    assert e.value.status == -1          # REVNET_E_INVALID_ARG
    B.revnet_check_device(ctx)
    r.load(inp["images"], inp["labels"], inp["params"])
    r.step()
    assert np.isfinite(r.results()["loss"])
    B.revnet_check_device(ctx)
    ctx.close()


def test_declared_buffers_smaller_than_planned_are_refused():
    ctx = B.Context(0)
    cfg = hp.tiny_stack("basic", N=8)
    inp = syn.make_stack_inputs(cfg)
    r = R.StackRunner(ctx, cfg, 0)
    r.load(inp["images"], inp["labels"], inp["params"])
    r.plan.set_buffer_sizes(r.plan.activation_bytes, r.plan.workspace_bytes - 1)
    with pytest.raises(B.RevnetError) as e:
        r.step()
    assert e.value.status == -3
    r.plan.set_buffer_sizes(r.act.numel(), r.ws.numel())
    r.step()
    assert np.isfinite(r.results()["loss"])
    ctx.close()


@pytest.mark.parametrize("use_graph", [False, True])
def test_timeline_mode_describes_the_last_step_and_changes_no_result(use_graph):
    """Timeline stamps: same bits as an unstamped step; every stamped launch has start <= end; the time with a
    stamped kernel running is no longer than the span from the first start to the last end."""
    ctx = B.Context(0)
    st = (syn.StageCfg(2, 64, 16, "bottleneck", 3, 1), syn.StageCfg(2, 128, 32, "bottleneck", 3, 2))
    cfg = syn.StackCfg("timeline", 8, 16, 10, 3, 1, 16, False, st, seed=5)
    inp = syn.make_stack_inputs(cfg)
    r = R.StackRunner(ctx, cfg, 0, use_cuda_graph=use_graph)
    got = []
    for stamped in (False, True, False):
        B.revnet_profile_enable(ctx, 3 if stamped else 0)
        r.load(inp["images"], inp["labels"], inp["params"])
        for _ in range(3):                      # under a graph: capture, then replays
            r.load(inp["images"], inp["labels"], inp["params"])
            st = r.step()
        torch.cuda.synchronize()
        got.append((float(r.loss.item()), r.params.cpu().numpy().copy()))
        if stamped:
            tl = B.revnet_profile_summary(ctx)
            span, busy = tl.pop("stamped_span"), tl.pop("stamped_busy")
            assert 0 < busy["ms"] <= span["ms"] * (1 + 1e-9)
            assert busy["launches"] == sum(v["launches"] for v in tl.values()) > 0
            assert busy["launches"] <= st.kernel_launches
            assert all(v["ms"] >= 0 and k.count("|") == 2 for k, v in tl.items())
            assert any(k.startswith("conv_") for k in tl) and any(k.startswith("bn_relu") for k in tl)
            assert span["ms"] < 1e3
    B.revnet_profile_enable(ctx, 0)
    for loss, params in got[1:]:
        assert loss == got[0][0] and np.array_equal(params, got[0][1])
    B.revnet_check_device(ctx)
    ctx.close()
