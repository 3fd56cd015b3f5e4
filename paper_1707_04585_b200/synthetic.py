"""Seeded synthetic workloads: network shapes and random inputs.

This module only describes shapes and draws random numbers.  It holds none of
the method's arithmetic, so that the CPU oracle and the CUDA path can both be
fed from it without sharing any computation.

Inputs stand in for CIFAR-10/100 and ImageNet batches: same tensor shapes
(3x32x32, 3x224x224; 10/100/1000 classes), values ~N(0,1), labels uniform.
Weights are Kaiming-normal (std = sqrt(2 / fan_in), fan_in = Cin*k*k), BN
affine parameters start at gamma=1, beta=0 (optionally jittered so that the
dgamma/dbeta paths see non-trivial values).

All arrays are "logical" NCHW / [Cout,Cin,kh,kw] float32; each consumer
converts to its own layout and precision.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Tuple

import numpy as np


@dataclass(frozen=True)
class StageCfg:
    units: int          # reversible units in this stage
    c: int              # channels per half (x1 and x2 each have c)
    w: int              # bottleneck width (0 for basic / single)
    kind: str           # "single" | "basic" | "bottleneck"
    trans_k: int        # kernel of the stored BN-ReLU-conv transition in front (0 = none)
    trans_stride: int   # its stride (1 = entry transition, 2 = down-sampling)
    down: bool = False  # paper-shaped stage: the first of its `units` units is a stored down-sampling unit
                        # (stride-2 layer inside F, shortcut skip paths) and trans_k is 0


@dataclass(frozen=True)
class StackCfg:
    name: str
    N: int
    img: int
    n_classes: int
    stem_k: int
    stem_stride: int
    stem_cout: int
    maxpool: bool
    stages: Tuple[StageCfg, ...]
    seed: int
    in_ch: int = 3
    eps: float = 1e-5
    lr: float = 0.1
    momentum: float = 0.9
    weight_decay: float = 2e-4

    @property
    def stem_pad(self) -> int:
        return self.stem_k // 2


@dataclass(frozen=True)
class BlockCfg:
    """A single reversible block (half-channels c, F and G of the same kind)."""
    N: int
    H: int
    W: int
    c: int
    w: int
    kind: str
    seed: int
    eps: float = 1e-5


def fn_layers(kind: str, c: int, w: int) -> List[Tuple[int, int, int]]:
    """(cin, cout, k) of each BN-ReLU-conv layer of a residual function."""
    if kind == "single":
        return [(c, c, 3)]
    if kind == "basic":
        return [(c, c, 3), (c, c, 3)]
    if kind == "bottleneck":
        return [(c, w, 1), (w, w, 3), (w, c, 1)]
    raise ValueError(kind)


def down_fn_layers(kind: str, cin_half: int, c: int, w: int) -> List[Tuple[int, int, int, int]]:
    """(cin, cout, k, stride) of the layers of F in a down-sampling unit: the stride sits on the first 3x3 of a basic
    function and on the 3x3 in the middle of a bottleneck; G of that unit is an ordinary stride-1 function."""
    if kind == "basic":
        return [(cin_half, c, 3, 2), (c, c, 3, 1)]
    if kind == "bottleneck":
        return [(cin_half, w, 1, 1), (w, w, 3, 2), (w, c, 1, 1)]
    raise ValueError(kind)


def reversible_units(s: StageCfg) -> int:
    return s.units - 1 if s.down else s.units


def _basic(units, cs):
    st = []
    for i, c in enumerate(cs):
        st.append(StageCfg(units, c, 0, "basic", 3 if i > 0 else 0, 2 if i > 0 else 1))
    return tuple(st)


def _bott(units, ws, first_entry=True):
    st = []
    for i, (u, w) in enumerate(zip(units, ws)):
        st.append(StageCfg(u, 4 * w, w, "bottleneck", 3, 2 if i > 0 else 1))
    return tuple(st)


def block_config_1() -> BlockCfg:
    return BlockCfg(N=4, H=8, W=8, c=8, w=0, kind="single", seed=0)


def stack_config(name: str) -> StackCfg:
    if name == "revnet38":
        return StackCfg("revnet38", 128, 32, 10, 3, 1, 32, False, _basic(3, (16, 32, 56)), seed=1)
    if name == "revnet110":
        return StackCfg("revnet110", 128, 32, 10, 3, 1, 32, False, _basic(9, (16, 32, 64)), seed=2)
    if name == "revnet164":
        return StackCfg("revnet164", 128, 32, 100, 3, 1, 32, False,
                        _bott((9, 9, 9), (32, 64, 128)), seed=3)
    if name == "revnet104":
        return StackCfg("revnet104", 64, 224, 1000, 7, 2, 128, True,
                        _bott((3, 4, 7, 3), (128, 256, 512, 832)), seed=4, weight_decay=1e-4)
    # Table "Architectural details" read with the down-sampling inside the first unit of stages 2.. (no separate
    # transitions): unit counts and stage widths as printed; for the bottleneck rows the per-half bottleneck widths
    # that come closest to the printed parameter counts
    if name == "paper_revnet38":
        return StackCfg(name, 128, 32, 10, 3, 1, 32, False, _paper("basic", (3, 3, 3), (16, 32, 56), (0, 0, 0)), seed=11)
    if name == "paper_revnet110":
        return StackCfg(name, 128, 32, 10, 3, 1, 32, False, _paper("basic", (9, 9, 9), (16, 32, 64), (0, 0, 0)), seed=12)
    if name == "paper_revnet164":
        return StackCfg(name, 128, 32, 10, 3, 1, 32, False, _paper("bottleneck", (9, 9, 9), (64, 128, 256), (16, 32, 64), entry=True), seed=13)
    if name == "paper_revnet104":
        return StackCfg(name, 64, 224, 1000, 7, 2, 128, True,
                        _paper("bottleneck", (2, 2, 11, 2), (256, 512, 1024, 1664), (64, 128, 256, 416), entry=True), seed=14, weight_decay=1e-4)
    raise ValueError(name)


def _paper(kind, units, cs, ws, entry=False):
    """Stages of a paper-shaped network: stage 0 starts from the stem (through a stored stride-1 entry layer where the
    stem's width differs from the stage's), later stages start with a down-sampling unit."""
    st = []
    for i, (u, c, w) in enumerate(zip(units, cs, ws)):
        if i == 0:
            st.append(StageCfg(u, c, w, kind, 3 if entry else 0, 1))
        else:
            st.append(StageCfg(u, c, w, kind, 0, 1, down=True))
    return tuple(st)


PAPER_NAMES = ("paper_revnet38", "paper_revnet110", "paper_revnet164", "paper_revnet104")
STACK_NAMES = ("revnet38", "revnet110", "revnet164", "revnet104")


def shrink(cfg: StackCfg, N: int = None, units: int = None, img: int = None) -> StackCfg:
    """Same widths, smaller batch / depth / image: for cases the oracle finishes quickly."""
    st = cfg.stages
    if units is not None:
        st = tuple(replace(s, units=units) for s in st)
    return replace(cfg, N=N or cfg.N, img=img or cfg.img, stages=st)


def stage_resolutions(cfg: StackCfg) -> List[int]:
    H = cfg.img // cfg.stem_stride
    if cfg.maxpool:
        H //= 2
    out = []
    for s in cfg.stages:
        if s.trans_k:
            H //= s.trans_stride
        if s.down:
            H //= 2
        out.append(H)
    return out


def param_specs(cfg: StackCfg) -> List[Tuple[str, Tuple[int, ...], str]]:
    """(name, shape, role) in forward order; role in {convw, gamma, beta, fcw, fcb}."""
    sp = [("stem.W", (cfg.stem_cout, cfg.in_ch, cfg.stem_k, cfg.stem_k), "convw")]
    cprev = cfg.stem_cout
    for si, s in enumerate(cfg.stages):
        if s.trans_k:
            sp += [(f"s{si}.T.gamma", (cprev,), "gamma"), (f"s{si}.T.beta", (cprev,), "beta"),
                   (f"s{si}.T.W", (2 * s.c, cprev, s.trans_k, s.trans_k), "convw")]
        elif s.down:
            for fn, layers in (("F", down_fn_layers(s.kind, cprev // 2, s.c, s.w)), ("G", fn_layers(s.kind, s.c, s.w))):
                for li, ly in enumerate(layers):
                    ci, co, k = ly[0], ly[1], ly[2]
                    p = f"s{si}.d.{fn}.l{li}"
                    sp += [(p + ".gamma", (ci,), "gamma"), (p + ".beta", (ci,), "beta"), (p + ".W", (co, ci, k, k), "convw")]
        else:
            assert cprev == 2 * s.c, "stage without transition must match incoming channels"
        for u in range(reversible_units(s)):
            for fn in "FG":
                for li, (ci, co, k) in enumerate(fn_layers(s.kind, s.c, s.w)):
                    p = f"s{si}.u{u}.{fn}.l{li}"
                    sp += [(p + ".gamma", (ci,), "gamma"), (p + ".beta", (ci,), "beta"),
                           (p + ".W", (co, ci, k, k), "convw")]
        cprev = 2 * s.c
    sp += [("fc.W", (cfg.n_classes, cprev), "fcw"), ("fc.b", (cfg.n_classes,), "fcb")]
    return sp


def block_param_specs(b: BlockCfg):
    sp = []
    for fn in "FG":
        for li, (ci, co, k) in enumerate(fn_layers(b.kind, b.c, b.w)):
            p = f"{fn}.l{li}"
            sp += [(p + ".gamma", (ci,), "gamma"), (p + ".beta", (ci,), "beta"),
                   (p + ".W", (co, ci, k, k), "convw")]
    return sp


def _draw_params(rng, specs, affine_jitter):
    out: Dict[str, np.ndarray] = {}
    for name, shape, role in specs:
        if role == "convw":
            fan_in = shape[1] * shape[2] * shape[3]
            out[name] = (rng.standard_normal(shape) * np.sqrt(2.0 / fan_in)).astype(np.float32)
        elif role == "fcw":
            out[name] = (rng.standard_normal(shape) * np.sqrt(2.0 / shape[1])).astype(np.float32)
        elif role == "fcb":
            out[name] = np.zeros(shape, np.float32)
        elif role == "gamma":
            g = 1.0 + (0.1 * rng.standard_normal(shape) if affine_jitter else 0.0)
            out[name] = np.broadcast_to(np.asarray(g, np.float32), shape).copy()
        elif role == "beta":
            b = 0.1 * rng.standard_normal(shape) if affine_jitter else 0.0
            out[name] = np.broadcast_to(np.asarray(b, np.float32), shape).copy()
    return out


def make_block_inputs(b: BlockCfg, affine_jitter: bool = False):
    """Draw order: x, then dy1, dy2, then weights in forward order (F then G)."""
    rng = np.random.Generator(np.random.PCG64(b.seed))
    x = rng.standard_normal((b.N, 2 * b.c, b.H, b.W)).astype(np.float32)
    dy1 = rng.standard_normal((b.N, b.c, b.H, b.W)).astype(np.float32)
    dy2 = rng.standard_normal((b.N, b.c, b.H, b.W)).astype(np.float32)
    params = _draw_params(rng, block_param_specs(b), affine_jitter)
    return dict(x1=x[:, :b.c].copy(), x2=x[:, b.c:].copy(), dy1=dy1, dy2=dy2, params=params)


def make_stack_inputs(cfg: StackCfg, affine_jitter: bool = False):
    """Draw order: images, labels, weights in forward order."""
    rng = np.random.Generator(np.random.PCG64(cfg.seed))
    images = rng.standard_normal((cfg.N, cfg.in_ch, cfg.img, cfg.img)).astype(np.float32)
    labels = rng.integers(0, cfg.n_classes, size=(cfg.N,)).astype(np.int32)
    params = _draw_params(rng, param_specs(cfg), affine_jitter)
    return dict(images=images, labels=labels, params=params)
