"""Parity at the real widths of the bottleneck configurations (BASELINE configs 4 and 5): blocks at
(c, w) = (512,128) ... (3328,832), the stored transitions 128->1024 (stride 1) ... 4096->6656
(stride 2), and one whole train step of the large-image network at its real widths and image size
with a small batch.  These shapes take the kernel paths the narrow cases never reach: many channel
chunks per tap, N tiles of 128 x 256, the ragged last N tile of 832 and 3328 channels, tiles that
hold several 7x7 images.  Forward outputs are held to the stated tolerance; gradients too, except
where tests/parity.py says beforehand that ReLU decisions are expected to differ (floor rule).
"""
import numpy as np
import pytest

from paper_1707_04585_b200 import binding as B
from paper_1707_04585_b200 import synthetic as syn
from tests import parity as par
from tests import test_gpu_parity as tp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    B.revnet_check_device(c)
    c.close()


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("N,H,c,w", [
    (2, 56, 512, 128),      # config 5, stage 1 (two image rows per tile)
    (2, 28, 1024, 256),     # stage 2 (112-pixel tiles)
    (2, 14, 2048, 512),     # stage 3 (one 14x14 image per tile is 196 pixels: ragged row tiles)
    (4, 7, 3328, 832),      # stage 4: two 7x7 images per tile, 832 = 6 x 128 + 64 and 3328 = 26 x 128 channels
    (3, 7, 3328, 832),      # ... and an odd batch: the last tile holds one image
    (8, 8, 512, 128),       # config 4, stage 3
])
def test_bottleneck_block_at_real_widths(ctx, mode, N, H, c, w):
    tp.run_block_case(ctx, syn.BlockCfg(N, H, H, c, w, "bottleneck", seed=500 + w), mode, jitter=True, inplace=True, tag=" wide")


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("N,H,cin,cout,stride,split", [
    (2, 56, 128, 1024, 1, False),    # config 5 entry transition behind the max-pool
    (2, 56, 1024, 2048, 2, True),
    (2, 28, 2048, 4096, 2, True),
    (2, 14, 4096, 6656, 2, True),    # 14x14 -> 7x7, 6656 = 52 x 128 output channels
    (4, 32, 32, 256, 1, False),      # config 4 entry transition
    (4, 16, 512, 1024, 2, True),     # config 4, last transition
])
def test_transition_at_real_widths(ctx, mode, N, H, cin, cout, stride, split):
    tp.run_transition_case(ctx, mode, N, H, cin, cout, 3, stride, split)


def test_revnet104_whole_step_real_widths_small_batch(ctx):
    """Config 5 as it is (7x7/2 stem, max-pool, widths 128/256/512/832, 224x224 images) at batch 2: the
    whole train step against the oracle; sampled units and all transitions inside the network at the
    stated tolerance or their own floor, end-to-end quantities by the floor rule."""
    cfg = syn.shrink(syn.stack_config("revnet104"), N=2)
    keys = ((0, 0), (1, 3), (2, 6), (3, 0), (3, 2))
    try:
        tp.run_blocks_in_network(ctx, cfg, 0, keys)
        tp.run_stack_case(ctx, cfg, 0, jitter=False, floor_levels=[2.0 ** -16], keep_blocks=keys, keep_transitions=True, logits_floor=True, floor_draws=1)
    finally:
        tp.ORACLE_RUNS.clear()
