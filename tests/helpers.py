"""Test-side glue: turn a synthetic config + parameter dict into the oracle's plain structures."""
import numpy as np

from paper_1707_04585_b200 import synthetic as syn


def oracle_fn(prefix, kind, c, w, params):
    return [dict(name=f"{prefix}.l{li}", gamma=params[f"{prefix}.l{li}.gamma"],
                 beta=params[f"{prefix}.l{li}.beta"], W=params[f"{prefix}.l{li}.W"])
            for li in range(len(syn.fn_layers(kind, c, w)))]


def oracle_block(b, params):
    return oracle_fn("F", b.kind, b.c, b.w, params), oracle_fn("G", b.kind, b.c, b.w, params)


def oracle_net(cfg, params):
    stages = []
    for si, s in enumerate(cfg.stages):
        trans = None
        if s.trans_k:
            trans = dict(name=f"s{si}.T", gamma=params[f"s{si}.T.gamma"], beta=params[f"s{si}.T.beta"],
                         W=params[f"s{si}.T.W"], stride=s.trans_stride)
        units = [(oracle_fn(f"s{si}.u{u}.F", s.kind, s.c, s.w, params),
                  oracle_fn(f"s{si}.u{u}.G", s.kind, s.c, s.w, params)) for u in range(syn.reversible_units(s))]
        down = None
        if s.down:
            cprev = cfg.stages[si - 1].c
            dF = [dict(name=f"s{si}.d.F.l{li}", gamma=params[f"s{si}.d.F.l{li}.gamma"], beta=params[f"s{si}.d.F.l{li}.beta"],
                       W=params[f"s{si}.d.F.l{li}.W"], stride=ly[3]) for li, ly in enumerate(syn.down_fn_layers(s.kind, cprev, s.c, s.w))]
            down = (dF, oracle_fn(f"s{si}.d.G", s.kind, s.c, s.w, params))
        stages.append(dict(trans=trans, down=down, c=s.c, units=units))
    return dict(stem=dict(name="stem", W=params["stem.W"], stride=cfg.stem_stride, pad=cfg.stem_pad),
                maxpool=cfg.maxpool, stages=stages,
                fc=dict(name="fc", W=params["fc.W"], b=params["fc.b"]), eps=cfg.eps)


def decayed_names(cfg):
    return {n for n, _, role in syn.param_specs(cfg) if role in ("convw", "fcw")}


def rel_l2(a, b):
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    d = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / d) if d > 0 else float(np.linalg.norm(a))


def tiny_stack(kind="basic", maxpool=False, N=4, img=8, units=2, seed=11, n_classes=5):
    """A few-thousand-parameter stack with every kind of layer the big configs have."""
    if kind == "basic":
        st = (syn.StageCfg(units, 4, 0, "basic", 0, 1), syn.StageCfg(units, 8, 0, "basic", 3, 2))
        stem_c = 8
    else:
        st = (syn.StageCfg(units, 8, 4, "bottleneck", 3, 1), syn.StageCfg(units, 12, 4, "bottleneck", 3, 2))
        stem_c = 8
    return syn.StackCfg(f"tiny_{kind}", N, img * (4 if maxpool else 1), n_classes,
                        7 if maxpool else 3, 2 if maxpool else 1, stem_c, maxpool, st, seed=seed)
