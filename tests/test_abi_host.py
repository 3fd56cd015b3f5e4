"""CPU-side checks of the C-ABI library: it loads, exports what the header declares, and its
planning logic (parameter layout, stored-activation accounting) is right.  No kernel runs here."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1707_04585_b200 import binding as B
from paper_1707_04585_b200 import build as libbuild
from paper_1707_04585_b200 import synthetic as syn
from oracle import revnet as orc
from tests import helpers as hp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ctx():
    libbuild.build()
    c = B.Context(device=-1)      # planning-only context: no CUDA call
    yield c
    c.close()


def test_library_exports_every_declared_symbol():
    libbuild.build()
    hdr = open(os.path.join(ROOT, "include", "revnet.h")).read()
    declared = set(re.findall(r"\b(revnet_[a-z_]+)\s*\(", hdr))
    assert declared == set(B.EXPORTS)
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("name", syn.STACK_NAMES)
def test_plan_parameter_count_matches_specs(ctx, name):
    cfg = syn.stack_config(name)
    plan = B.revnet_stack_plan(ctx, B.stack_desc(cfg, 0))
    assert plan.param_count == sum(int(np.prod(s)) for _, s, _ in syn.param_specs(cfg))
    plan.close()


def test_activation_bytes_flat_in_depth_and_equal_to_oracle_count(ctx):
    base = syn.stack_config("revnet110")
    sizes = {}

    def pad(n): return (n + 255) // 256 * 256

    def scratch(plan, cfg):
        # the workspace also carries per-parameter data (bf16 weight packs, SGD segment table), which
        # grows with depth like the parameters do; the activation scratch must not
        assert plan.param_scratch_bytes + plan.activation_scratch_bytes == plan.workspace_bytes
        return plan.activation_scratch_bytes
    for units in (1, 3, 9, 18, 36):
        cfg = syn.shrink(base, units=units)
        plan = B.revnet_stack_plan(ctx, B.stack_desc(cfg, 0))
        sizes[units] = (plan.activation_bytes, scratch(plan, cfg))
        plan.close()
    assert len(set(sizes.values())) == 1, sizes           # integer equality across depths (Section 3.2)
    base = syn.stack_config("revnet164")
    s164 = set()
    for units in (1, 9, 36):
        cfg = syn.shrink(base, units=units)
        plan = B.revnet_stack_plan(ctx, B.stack_desc(cfg, 0))
        s164.add((plan.activation_bytes, scratch(plan, cfg))); plan.close()
    assert len(s164) == 1


@pytest.mark.parametrize("kind,maxpool", [("basic", False), ("bottleneck", False), ("bottleneck", True)])
def test_stored_bytes_equal_oracle_accounting(ctx, kind, maxpool):
    """The oracle counts what its reconstructing pass keeps; the plan must keep exactly that."""
    cfg = hp.tiny_stack(kind, maxpool)
    inp = syn.make_stack_inputs(cfg)
    r = orc.stack_train_grads(hp.oracle_net(cfg, inp["params"]), inp["images"], inp["labels"], "reconstruct")
    plan = B.revnet_stack_plan(ctx, B.stack_desc(cfg, 1))
    images_bytes = inp["images"].size * 4
    # activation_bytes is 256-byte padded per tensor; compare against the padded oracle figure
    def pad(n): return (n + 255) // 256 * 256
    H = syn.stage_resolutions(cfg)
    expect = 0
    if cfg.maxpool or cfg.stages[0].trans_k:
        hs = cfg.img // cfg.stem_stride
        expect += pad(cfg.N * hs * hs * cfg.stem_cout * 4)
        if cfg.maxpool:
            expect += pad(cfg.N * (hs // 2) ** 2 * cfg.stem_cout * 4)
    for s, h in zip(cfg.stages, H):
        expect += 2 * pad(cfg.N * h * h * s.c * 4)
    assert plan.activation_bytes == expect
    unpadded = expect  # tiny tensors here are multiples of 256 bytes or padded; check against oracle when exact
    sizes = [cfg.N * h * h * s.c * 4 for s, h in zip(cfg.stages, H)]
    if all(x % 256 == 0 for x in sizes):
        assert r["stored_bytes"] == images_bytes + unpadded
    plan.close()


def test_bad_descriptors_are_rejected(ctx):
    cfg = syn.stack_config("revnet38")
    d = B.stack_desc(cfg, 0)
    d.stage[1].c = 30                      # not a multiple of 4
    with pytest.raises(B.RevnetError):
        B.revnet_stack_plan(ctx, d)
    d = B.stack_desc(cfg, 0); d.mode = 7
    with pytest.raises(B.RevnetError):
        B.revnet_stack_plan(ctx, d)
    bd = B.block_desc(syn.block_config_1(), 1); bd.G.cout[0] = 12
    with pytest.raises(B.RevnetError):
        B.revnet_block_workspace_bytes(ctx, bd)


def test_pack_bytes_and_declared_buffer_sizes(ctx):
    """Host logic of the pre-packed weights and of the declared buffer sizes (no kernel runs)."""
    b = syn.BlockCfg(2, 8, 8, 128, 32, "bottleneck", seed=1)
    n0 = B.revnet_block_pack_bytes(ctx, B.block_desc(b, 0, 16))
    # two packs (forward, data gradient) of cout x taps x cin bf16 per layer, rows and columns padded to 16, 256-byte slots
    expect = 0
    for (ci, co, k) in syn.fn_layers(b.kind, b.c, b.w) * 2:
        expect += 2 * ((co * k * k * ci * 2 + 255) // 256 * 256)
    assert n0 == expect
    assert B.revnet_block_pack_bytes(ctx, B.block_desc(b, 1, 0)) == 0          # strict fp32 mode has no packs
    odd = syn.BlockCfg(2, 8, 8, 12, 0, "basic", seed=1)                        # 12 channels: the fp32 kernels take it, no pack
    assert B.revnet_block_pack_bytes(ctx, B.block_desc(odd, 0, 16)) == 0
    cfg = hp.tiny_stack("basic")
    plan = B.revnet_stack_plan(ctx, B.stack_desc(cfg, 0))
    plan.set_buffer_sizes(plan.activation_bytes, plan.workspace_bytes)
    plan.close()
