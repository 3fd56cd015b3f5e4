"""Convenience wrappers that own the device buffers of one block / one stack and call the C ABI.

Marshalling only: numpy (NCHW, [Cout,Cin,kh,kw]) in, torch CUDA buffers in the ABI's layouts,
numpy out.  Used by the tests, the smoke check and the benchmark.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import synthetic as syn


def _dev(a, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dtype).cuda()


DEFAULT_FRAC_BITS = {0: 16, 1: 0}   # bf16 mode runs on the exactly invertible fixed-point state


def to_state(x_nchw: np.ndarray, frac_bits: int):
    """NCHW float array -> device NHWC tensor in the state format (float32, or int32 fixed point)."""
    x = B.to_nhwc(np.asarray(x_nchw, np.float32))
    if frac_bits == 0:
        return torch.from_numpy(x).cuda()
    return torch.from_numpy(np.rint(x.astype(np.float64) * (1 << frac_bits)).astype(np.int32)).cuda()


def from_state(t: torch.Tensor, frac_bits: int) -> np.ndarray:
    """device NHWC state tensor -> NCHW float64 array (exact for fixed point)."""
    a = t.cpu().numpy()
    a = a.astype(np.float64) if frac_bits == 0 else a.astype(np.float64) / (1 << frac_bits)
    return B.to_nchw(a)


class BlockRunner:
    def __init__(self, ctx: B.Context, b: syn.BlockCfg, mode: int, frac_bits: int = None):
        self.ctx, self.b, self.mode = ctx, b, mode
        self.frac = DEFAULT_FRAC_BITS[mode] if frac_bits is None else frac_bits
        self.desc = B.block_desc(b, mode, self.frac)
        fwd, bwd = B.revnet_block_workspace_bytes(ctx, self.desc)
        self.ws = torch.empty(max(fwd, bwd), dtype=torch.uint8, device="cuda")
        self.layers = syn.fn_layers(b.kind, b.c, b.w)

    def _params(self, params, fn):
        return [dict(W=_dev(B.w_to_abi(params[f"{fn}.l{i}.W"])), gamma=_dev(params[f"{fn}.l{i}.gamma"]),
                     beta=_dev(params[f"{fn}.l{i}.beta"])) for i in range(len(self.layers))]

    def load(self, params):
        self.F, self.G = self._params(params, "F"), self._params(params, "G")
        self.gF = [{k: torch.zeros_like(v) for k, v in l.items()} for l in self.F]
        self.gG = [{k: torch.zeros_like(v) for k, v in l.items()} for l in self.G]
        self.packs = None

    def pack(self):
        """Build the bf16 weight packs once (revnet_pack_weights); later calls reuse them."""
        n = B.revnet_block_pack_bytes(self.ctx, self.desc)
        self.packs = torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")
        B.revnet_pack_weights(self.ctx, self.desc, self.F, self.G, self.packs)

    def forward(self, x1, x2, inplace=False):
        """x1, x2: NCHW numpy -> y1, y2 NCHW numpy (values of the state format, exact)"""
        dx1, dx2 = to_state(x1, self.frac), to_state(x2, self.frac)
        y1, y2 = (dx1, dx2) if inplace else (torch.empty_like(dx1), torch.empty_like(dx2))
        B.revnet_block_fwd(self.ctx, self.desc, dx1, dx2, self.F, self.G, y1, y2, self.ws)
        torch.cuda.synchronize()
        return from_state(y1, self.frac), from_state(y2, self.frac)

    def backward(self, y1, y2, dy1, dy2, inplace=False):
        ty1, ty2 = to_state(y1, self.frac), to_state(y2, self.frac)
        tdy1, tdy2 = (_dev(B.to_nhwc(t)) for t in (dy1, dy2))
        if inplace:
            x1, x2, dx1, dx2 = ty1, ty2, tdy1, tdy2
        else:
            x1, x2 = torch.empty_like(ty1), torch.empty_like(ty2)
            dx1, dx2 = torch.empty_like(tdy1), torch.empty_like(tdy2)
        B.revnet_block_bwd(self.ctx, self.desc, ty1, ty2, tdy1, tdy2, self.F, self.G, x1, x2, dx1, dx2, self.gF, self.gG, self.ws)
        torch.cuda.synchronize()
        grads = {}
        for fn, gl in (("F", self.gF), ("G", self.gG)):
            for i, l in enumerate(gl):
                grads[f"{fn}.l{i}.W"] = B.w_from_abi(l["W"].cpu().numpy())
                grads[f"{fn}.l{i}.gamma"] = l["gamma"].cpu().numpy()
                grads[f"{fn}.l{i}.beta"] = l["beta"].cpu().numpy()
        return (from_state(x1, self.frac), from_state(x2, self.frac),
                B.to_nchw(dx1.cpu().numpy()), B.to_nchw(dx2.cpu().numpy()), grads)


class StackRunner:
    def __init__(self, ctx: B.Context, cfg: syn.StackCfg, mode: int, verify_reconstruction: bool = False,
                 frac_bits: int = None, use_cuda_graph: bool = True, store_activations: bool = False):
        self.ctx, self.cfg, self.mode = ctx, cfg, mode
        self.frac = DEFAULT_FRAC_BITS[mode] if frac_bits is None else frac_bits
        self.specs = syn.param_specs(cfg)
        self.desc = B.stack_desc(cfg, mode, verify_reconstruction, self.frac, use_cuda_graph, store_activations)
        self.plan = B.revnet_stack_plan(ctx, self.desc)
        n = self.plan.param_count
        assert n == sum(int(np.prod(s)) for _, s, _ in self.specs)
        self.params = torch.zeros(n, dtype=torch.float32, device="cuda")
        self.grads = torch.zeros(n, dtype=torch.float32, device="cuda")
        self.momentum = torch.zeros(n, dtype=torch.float32, device="cuda")
        self.act = torch.empty(self.plan.activation_bytes, dtype=torch.uint8, device="cuda")
        self.ws = torch.empty(self.plan.workspace_bytes, dtype=torch.uint8, device="cuda")
        self.images = torch.empty((cfg.N, cfg.img, cfg.img, cfg.in_ch), dtype=torch.float32, device="cuda")
        self.labels = torch.empty((cfg.N,), dtype=torch.int32, device="cuda")
        self.loss = torch.zeros(1, dtype=torch.float32, device="cuda")
        self.pred = torch.zeros(cfg.N, dtype=torch.int32, device="cuda")
        self.logits = torch.zeros((cfg.N, cfg.n_classes), dtype=torch.float32, device="cuda")

    def load(self, images, labels, params):
        self.images.copy_(torch.from_numpy(B.to_nhwc(images)))
        self.labels.copy_(torch.from_numpy(np.asarray(labels, np.int32)))
        self.params.copy_(torch.from_numpy(B.pack_params(self.specs, params)))
        self.momentum.zero_()

    def step(self, want_logits=True):
        return B.revnet_train_step(self.ctx, self.plan, self.images, self.labels, self.params, self.grads, self.momentum,
                                   self.act, self.ws, self.loss, self.pred, self.logits if want_logits else None)

    def results(self):
        torch.cuda.synchronize()
        return dict(loss=float(self.loss.item()), pred=self.pred.cpu().numpy(), logits=self.logits.cpu().numpy(),
                    grads=B.unpack_params(self.specs, self.grads.cpu().numpy()),
                    params=B.unpack_params(self.specs, self.params.cpu().numpy()),
                    momentum=B.unpack_params(self.specs, self.momentum.cpu().numpy()))


def time_block(ctx: B.Context, b: syn.BlockCfg, mode: int, reps: int = 10, warmup: int = 3, graph: bool = True):
    """Device time (ms) of one block forward and one reconstructing backward at shape b, in place,
    through the C ABI, with CUDA events on the launching stream.  With graph=True each of the two
    calls is captured once into a CUDA graph and replayed, so the figure holds kernel time without
    the host's launch overhead (as in a train step, which replays a graph too)."""
    inp = syn.make_block_inputs(b, affine_jitter=True)
    r = BlockRunner(ctx, b, mode)
    r.load(inp["params"])
    r.pack()        # as in a train step, the weight packs exist before the block runs: the times hold the block alone
    x1, x2 = to_state(inp["x1"], r.frac), to_state(inp["x2"], r.frac)
    d1, d2 = _dev(B.to_nhwc(inp["dy1"])), _dev(B.to_nhwc(inp["dy2"]))

    def fwd():
        B.revnet_block_fwd(ctx, r.desc, x1, x2, r.F, r.G, x1, x2, r.ws)

    def bwd():
        B.revnet_block_bwd(ctx, r.desc, x1, x2, d1, d2, r.F, r.G, x1, x2, d1, d2, r.gF, r.gG, r.ws)

    fwd(); bwd()                      # first-call set-up happens outside any capture
    torch.cuda.synchronize()
    if graph:
        side = torch.cuda.Stream()
        graphs = []
        for fn in (fwd, bwd):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    fn()
            graphs.append(g)
        torch.cuda.synchronize()
        run_f, run_b = graphs[0].replay, graphs[1].replay
    else:
        run_f, run_b = fwd, bwd
    stream = torch.cuda.current_stream()
    ms = {"fwd": [], "bwd": []}
    for i in range(warmup + reps):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record(stream)
        run_f()
        e[1].record(stream)
        run_b()
        e[2].record(stream)
        torch.cuda.synchronize()
        if i >= warmup:
            ms["fwd"].append(e[0].elapsed_time(e[1])); ms["bwd"].append(e[1].elapsed_time(e[2]))
    B.revnet_check_device(ctx)
    return {k: float(np.median(v)) for k, v in ms.items()}


def time_transition(ctx: B.Context, N: int, H: int, cin: int, cout: int, k: int, stride: int, split: bool, mode: int,
                    reps: int = 10, warmup: int = 3):
    """Device time (ms) of one stored BN-ReLU-conv layer, forward and backward, through the C ABI."""
    frac = DEFAULT_FRAC_BITS[mode]
    rng = np.random.default_rng(5)
    d = B.TransitionDesc(N, H, H, cin, cout, k, stride, int(split), 1e-5, mode, frac)
    fb, bb = B.revnet_transition_workspace_bytes(ctx, d)
    ws = torch.empty(max(fb, bb), dtype=torch.uint8, device="cuda")
    Ho = H // stride
    rand = lambda *sh: torch.from_numpy(rng.standard_normal(sh).astype(np.float32)).cuda()
    if split:
        x = rng.standard_normal((N, cin, H, H)).astype(np.float32)
        in1, in2 = to_state(x[:, :cin // 2], frac), to_state(x[:, cin // 2:], frac)
        di1, di2 = torch.empty((N, H, H, cin // 2), dtype=torch.float32, device="cuda"), torch.empty((N, H, H, cin // 2), dtype=torch.float32, device="cuda")
    else:
        in1, in2, di1, di2 = rand(N, H, H, cin), None, torch.empty((N, H, H, cin), dtype=torch.float32, device="cuda"), None
    W = rand(cout, k, k, cin) * float(np.sqrt(2.0 / (cin * k * k)))
    g, b_ = torch.ones(cin, device="cuda"), torch.zeros(cin, device="cuda")
    o1 = torch.empty((N, Ho, Ho, cout // 2), dtype=torch.int32 if frac else torch.float32, device="cuda"); o2 = torch.empty_like(o1)
    d1, d2 = rand(N, Ho, Ho, cout // 2), rand(N, Ho, Ho, cout // 2)
    gW, gg, gb = torch.empty_like(W), torch.empty_like(g), torch.empty_like(b_)
    stream = torch.cuda.current_stream()
    ms = {"fwd": [], "bwd": []}
    for i in range(warmup + reps):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record(stream)
        B.revnet_transition_fwd(ctx, d, in1, in2, W, g, b_, o1, o2, ws)
        e[1].record(stream)
        B.revnet_transition_bwd(ctx, d, in1, in2, d1, d2, W, g, b_, di1, di2, gW, gg, gb, ws)
        e[2].record(stream)
        torch.cuda.synchronize()
        if i >= warmup:
            ms["fwd"].append(e[0].elapsed_time(e[1])); ms["bwd"].append(e[1].elapsed_time(e[2]))
    B.revnet_check_device(ctx)
    return {k_: float(np.median(v)) for k_, v in ms.items()}


if __name__ == "__main__":
    import argparse, json
    ap = argparse.ArgumentParser(description="time one reversible block (forward, reconstructing backward), or one stored transition layer")
    ap.add_argument("--trans", default="", help="cin,cout,stride[,split]: time a stored 3x3 BN-ReLU-conv layer on an HxH input instead of a block")
    ap.add_argument("--N", type=int, default=128); ap.add_argument("--H", type=int, default=32)
    ap.add_argument("--c", type=int, default=64); ap.add_argument("--w", type=int, default=0)
    ap.add_argument("--kind", default="basic"); ap.add_argument("--mode", type=int, default=0)
    ap.add_argument("--reps", type=int, default=10); ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--eager", action="store_true", help="launch kernel by kernel instead of replaying CUDA graphs")
    a = ap.parse_args()
    c = B.Context(0)
    if a.trans:
        t = [int(v) for v in a.trans.split(",")]
        print(json.dumps(dict(shape=vars(a), ms=time_transition(c, a.N, a.H, t[0], t[1], 3, t[2], bool(t[3]) if len(t) > 3 else t[2] == 2, a.mode, a.reps, a.warmup))))
        raise SystemExit(0)
    print(json.dumps(dict(shape=vars(a), ms=time_block(c, syn.BlockCfg(a.N, a.H, a.H, a.c, a.w, a.kind, seed=5), a.mode, a.reps, a.warmup, graph=not a.eager))))
