"""ctypes binding of librevnet.so: argument marshalling only.

Every function mirrors the C entry point of the same name (include/revnet.h) and takes torch
CUDA tensors (for their device pointers) or raw integers.  No arithmetic of the method happens
here; the layout helpers only permute / concatenate arrays into the ABI's layouts.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List

import numpy as np

from . import synthetic as syn

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librevnet.so")
MAX_STAGES = 8
_lib = None

EXPORTS = ["revnet_create", "revnet_destroy", "revnet_last_error", "revnet_block_workspace_bytes",
           "revnet_block_fwd", "revnet_block_bwd", "revnet_stack_plan", "revnet_plan_destroy",
           "revnet_train_step", "revnet_train_step_host", "revnet_profile_enable", "revnet_profile_summary", "revnet_check_device", "revnet_plan_scratch_split",
           "revnet_transition_workspace_bytes", "revnet_transition_fwd", "revnet_transition_bwd",
           "revnet_block_fwd_noalloc", "revnet_block_pack_bytes", "revnet_pack_weights", "revnet_selftest_bounded_wait",
           "revnet_plan_set_buffer_sizes"]


class FnDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("k", C.c_int * 3), ("cin", C.c_int * 3), ("cout", C.c_int * 3)]


class BlockDesc(C.Structure):
    _fields_ = [("N", C.c_int), ("H", C.c_int), ("W", C.c_int), ("c", C.c_int), ("F", FnDesc), ("G", FnDesc),
                ("eps", C.c_float), ("mode", C.c_int), ("state_frac_bits", C.c_int)]


class FnParams(C.Structure):
    _fields_ = [("W", C.c_void_p * 3), ("gamma", C.c_void_p * 3), ("beta", C.c_void_p * 3),
                ("Wpack_fprop", C.c_void_p * 3), ("Wpack_dgrad", C.c_void_p * 3)]


class FnGrads(C.Structure):
    _fields_ = [("dW", C.c_void_p * 3), ("dgamma", C.c_void_p * 3), ("dbeta", C.c_void_p * 3)]


class TransitionDesc(C.Structure):
    _fields_ = [("N", C.c_int), ("H", C.c_int), ("W", C.c_int), ("cin", C.c_int), ("cout", C.c_int), ("k", C.c_int),
                ("stride", C.c_int), ("in_split", C.c_int), ("eps", C.c_float), ("mode", C.c_int), ("state_frac_bits", C.c_int)]


class StageDesc(C.Structure):
    _fields_ = [("units", C.c_int), ("c", C.c_int), ("w", C.c_int), ("kind", C.c_int), ("trans_k", C.c_int),
                ("trans_stride", C.c_int), ("down", C.c_int)]


class StackDesc(C.Structure):
    _fields_ = [("N", C.c_int), ("img", C.c_int), ("in_ch", C.c_int), ("n_classes", C.c_int),
                ("stem_k", C.c_int), ("stem_stride", C.c_int), ("stem_cout", C.c_int), ("maxpool", C.c_int),
                ("n_stages", C.c_int), ("stage", StageDesc * MAX_STAGES), ("eps", C.c_float), ("mode", C.c_int),
                ("state_frac_bits", C.c_int), ("lr", C.c_float), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("verify_reconstruction", C.c_int), ("use_cuda_graph", C.c_int), ("store_activations", C.c_int)]


class StepStats(C.Structure):
    _fields_ = [("stored_activation_bytes", C.c_uint64), ("workspace_peak_bytes", C.c_uint64),
                ("flops_fwd", C.c_uint64), ("flops_bwd", C.c_uint64), ("kernel_launches", C.c_uint64),
                ("recon_max_abs", C.c_float * MAX_STAGES), ("device_status", C.c_int)]


def lib():
    """Load the CUDA library; there is no fallback if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1707_04585_b200.build`; "
                               "there is no CPU fallback")
        _lib = C.CDLL(LIB_PATH)
        _lib.revnet_last_error.restype = C.c_char_p
        _lib.revnet_last_error.argtypes = [C.c_void_p]
        for name in EXPORTS:
            if name != "revnet_last_error":
                getattr(_lib, name).restype = C.c_int
    return _lib


class RevnetError(RuntimeError):
    status = 0          # the revnet_status the call returned


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, int):
        return C.c_void_p(t)
    return C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Context:
    def __init__(self, device: int = 0):
        self.h = C.c_void_p()
        rc = lib().revnet_create(C.byref(self.h), C.c_int(device))
        if rc:
            raise RevnetError(f"revnet_create failed ({rc})")

    def check(self, rc, what):
        if rc:
            e = RevnetError(f"{what}: status {rc}: {lib().revnet_last_error(self.h).decode()}")
            e.status = rc
            raise e

    def close(self):
        if self.h:
            lib().revnet_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


KIND = {"single": 0, "basic": 1, "bottleneck": 2}


def fn_desc(kind: str, c: int, w: int) -> FnDesc:
    d = FnDesc()
    ls = syn.fn_layers(kind, c, w)
    d.n_layers = len(ls)
    for i, (ci, co, k) in enumerate(ls):
        d.cin[i], d.cout[i], d.k[i] = ci, co, k
    return d


def block_desc(b: syn.BlockCfg, mode: int, state_frac_bits: int = 0) -> BlockDesc:
    d = BlockDesc()
    d.N, d.H, d.W, d.c = b.N, b.H, b.W, b.c
    d.F = fn_desc(b.kind, b.c, b.w)
    d.G = fn_desc(b.kind, b.c, b.w)
    d.eps, d.mode, d.state_frac_bits = b.eps, mode, state_frac_bits
    return d


def stack_desc(cfg: syn.StackCfg, mode: int, verify_reconstruction: bool = False, state_frac_bits: int = 0,
               use_cuda_graph: bool = True, store_activations: bool = False) -> StackDesc:
    d = StackDesc()
    d.N, d.img, d.in_ch, d.n_classes = cfg.N, cfg.img, cfg.in_ch, cfg.n_classes
    d.stem_k, d.stem_stride, d.stem_cout, d.maxpool = cfg.stem_k, cfg.stem_stride, cfg.stem_cout, int(cfg.maxpool)
    d.n_stages = len(cfg.stages)
    for i, s in enumerate(cfg.stages):
        d.stage[i] = StageDesc(s.units, s.c, s.w, KIND[s.kind], s.trans_k, s.trans_stride, int(s.down))
    d.eps, d.mode, d.state_frac_bits = cfg.eps, mode, state_frac_bits
    d.lr, d.momentum, d.weight_decay = cfg.lr, cfg.momentum, cfg.weight_decay
    d.verify_reconstruction = int(verify_reconstruction)
    d.use_cuda_graph = int(use_cuda_graph)
    d.store_activations = int(store_activations)
    return d


# ------------------------------------------------------------------ layout helpers (no arithmetic)
def to_nhwc(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(np.transpose(x, (0, 2, 3, 1)))


def to_nchw(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(np.transpose(x, (0, 3, 1, 2)))


def w_to_abi(w: np.ndarray) -> np.ndarray:
    """[Cout,Cin,kh,kw] -> [Cout,kh,kw,Cin]"""
    return np.ascontiguousarray(np.transpose(w, (0, 2, 3, 1)))


def w_from_abi(w: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(np.transpose(w, (0, 3, 1, 2)))


def pack_params(specs, params: Dict[str, np.ndarray]) -> np.ndarray:
    """Flat float32 buffer in the ABI's parameter order (forward order)."""
    parts = []
    for name, shape, role in specs:
        a = np.asarray(params[name], np.float32)
        parts.append((w_to_abi(a) if role == "convw" else a).ravel())
    return np.concatenate(parts)


def unpack_params(specs, flat: np.ndarray) -> Dict[str, np.ndarray]:
    out, o = {}, 0
    for name, shape, role in specs:
        n = int(np.prod(shape))
        a = np.asarray(flat[o:o + n])
        if role == "convw":
            co, ci, kh, kw = shape
            a = w_from_abi(a.reshape(co, kh, kw, ci))
        else:
            a = a.reshape(shape)
        out[name] = a
        o += n
    assert o == flat.size
    return out


# ------------------------------------------------------------------ block-level calls
def revnet_block_workspace_bytes(ctx: Context, desc: BlockDesc):
    f, b = C.c_size_t(), C.c_size_t()
    ctx.check(lib().revnet_block_workspace_bytes(ctx.h, C.byref(desc), C.byref(f), C.byref(b)), "revnet_block_workspace_bytes")
    return f.value, b.value


def _fn_params(tensors: List[dict]) -> FnParams:
    """Layer dicts -> the ABI struct.  Optional integer entries "Wpack_fprop" / "Wpack_dgrad" (device
    addresses written by revnet_pack_weights) are passed through."""
    p = FnParams()
    for i, t in enumerate(tensors):
        p.W[i], p.gamma[i], p.beta[i] = t["W"].data_ptr(), t["gamma"].data_ptr(), t["beta"].data_ptr()
        p.Wpack_fprop[i], p.Wpack_dgrad[i] = t.get("Wpack_fprop") or None, t.get("Wpack_dgrad") or None
    return p


def revnet_block_pack_bytes(ctx, desc) -> int:
    n = C.c_size_t()
    ctx.check(lib().revnet_block_pack_bytes(ctx.h, C.byref(desc), C.byref(n)), "revnet_block_pack_bytes")
    return n.value


def revnet_pack_weights(ctx, desc, F, G, pack_buffer):
    """Build the bf16 weight packs of a block into pack_buffer and record their addresses in the layer
    dicts of F and G (keys "Wpack_fprop", "Wpack_dgrad"); later block calls with these dicts use them."""
    fp, gp = _fn_params(F), _fn_params(G)
    ctx.check(lib().revnet_pack_weights(ctx.h, C.byref(desc), C.byref(fp), C.byref(gp), _ptr(pack_buffer),
                                        C.c_size_t(pack_buffer.numel() * pack_buffer.element_size()), _stream()), "revnet_pack_weights")
    for st, layers in ((fp, F), (gp, G)):
        for i, t in enumerate(layers):
            t["Wpack_fprop"], t["Wpack_dgrad"] = st.Wpack_fprop[i], st.Wpack_dgrad[i]


def _fn_grads(tensors: List[dict]) -> FnGrads:
    g = FnGrads()
    for i, t in enumerate(tensors):
        g.dW[i], g.dgamma[i], g.dbeta[i] = t["W"].data_ptr(), t["gamma"].data_ptr(), t["beta"].data_ptr()
    return g


def revnet_block_fwd(ctx, desc, x1, x2, F, G, y1, y2, workspace):
    fp, gp = _fn_params(F), _fn_params(G)
    ctx.check(lib().revnet_block_fwd(ctx.h, C.byref(desc), _ptr(x1), _ptr(x2), C.byref(fp), C.byref(gp), _ptr(y1), _ptr(y2),
                                     _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()), _stream()),
              "revnet_block_fwd")


def revnet_block_bwd(ctx, desc, y1, y2, dy1, dy2, F, G, x1, x2, dx1, dx2, gF, gG, workspace):
    fp, gp, fg, gg = _fn_params(F), _fn_params(G), _fn_grads(gF), _fn_grads(gG)
    ctx.check(lib().revnet_block_bwd(ctx.h, C.byref(desc), _ptr(y1), _ptr(y2), _ptr(dy1), _ptr(dy2), C.byref(fp), C.byref(gp),
                                     _ptr(x1), _ptr(x2), _ptr(dx1), _ptr(dx2), C.byref(fg), C.byref(gg),
                                     _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()), _stream()),
              "revnet_block_bwd")


# ------------------------------------------------------------------ stack-level calls
class Plan:
    def __init__(self, ctx: Context, desc: StackDesc):
        self.ctx, self.desc = ctx, desc
        self.h = C.c_void_p()
        n, a, w = C.c_size_t(), C.c_size_t(), C.c_size_t()
        ctx.check(lib().revnet_stack_plan(ctx.h, C.byref(desc), C.byref(self.h), C.byref(n), C.byref(a), C.byref(w)),
                  "revnet_stack_plan")
        self.param_count, self.activation_bytes, self.workspace_bytes = n.value, a.value, w.value
        ps, as_ = C.c_size_t(), C.c_size_t()
        ctx.check(lib().revnet_plan_scratch_split(self.h, C.byref(ps), C.byref(as_)), "revnet_plan_scratch_split")
        self.param_scratch_bytes, self.activation_scratch_bytes = ps.value, as_.value

    def set_buffer_sizes(self, activation_bytes: int, workspace_bytes: int):
        self.ctx.check(lib().revnet_plan_set_buffer_sizes(self.h, C.c_size_t(activation_bytes), C.c_size_t(workspace_bytes)),
                       "revnet_plan_set_buffer_sizes")

    def close(self):
        if self.h:
            lib().revnet_plan_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def revnet_stack_plan(ctx: Context, desc: StackDesc) -> Plan:
    return Plan(ctx, desc)


def revnet_train_step(ctx, plan, images, labels, params, grads, momentum, activations, workspace, loss, pred,
                      logits=None, want_stats=True):
    st = StepStats()
    ctx.check(lib().revnet_train_step(ctx.h, plan.h, _ptr(images), _ptr(labels), _ptr(params), _ptr(grads), _ptr(momentum),
                                      _ptr(activations), _ptr(workspace), _ptr(loss), _ptr(pred), _ptr(logits),
                                      C.byref(st) if want_stats else C.c_void_p(0), _stream()), "revnet_train_step")
    return st


def revnet_train_step_host(ctx, plan, images_host, labels_host, images_dev, labels_dev, params, grads, momentum,
                           activations, workspace, loss_dev, pred_dev, loss_host, pred_host):
    """images_host / labels_host / loss_host / pred_host: CPU tensors (pinned recommended)."""
    st = StepStats()
    ctx.check(lib().revnet_train_step_host(ctx.h, plan.h, _ptr(images_host), _ptr(labels_host), _ptr(images_dev),
                                           _ptr(labels_dev), _ptr(params), _ptr(grads), _ptr(momentum), _ptr(activations),
                                           _ptr(workspace), _ptr(loss_dev), _ptr(pred_dev), _ptr(loss_host), _ptr(pred_host),
                                           C.byref(st), _stream()), "revnet_train_step_host")
    return st


def revnet_profile_enable(ctx, on):
    """0 / False: off; 1 / True: one record per kernel name; 2: one per kernel name and launch shape;
    3: timeline of the last train step from start / end stamps the kernels write themselves (no events)."""
    ctx.check(lib().revnet_profile_enable(ctx.h, C.c_int(int(on))), "revnet_profile_enable")


def revnet_profile_summary(ctx):
    """-> {kernel name: dict(launches, ms, bytes, flops)}"""
    need = C.c_size_t()
    ctx.check(lib().revnet_profile_summary(ctx.h, None, C.c_size_t(0), C.byref(need)), "revnet_profile_summary")
    buf = C.create_string_buffer(need.value + 16)
    ctx.check(lib().revnet_profile_summary(ctx.h, buf, C.c_size_t(need.value + 16), None), "revnet_profile_summary")
    out = {}
    for line in buf.value.decode().splitlines():
        name, n, ms, by, fl = line.split("\t")
        out[name] = dict(launches=int(n), ms=float(ms), bytes=float(by), flops=float(fl))
    return out


def revnet_check_device(ctx):
    """Synchronise and raise if a kernel reported that it gave up a bounded wait."""
    ctx.check(lib().revnet_check_device(ctx.h, _stream()), "revnet_check_device")


def revnet_selftest_bounded_wait(ctx, limit_ns: int):
    ctx.check(lib().revnet_selftest_bounded_wait(ctx.h, C.c_uint64(limit_ns), _stream()), "revnet_selftest_bounded_wait")


def _nbytes(t):
    return C.c_size_t(t.numel() * t.element_size())


def revnet_transition_workspace_bytes(ctx, desc):
    f, b = C.c_size_t(), C.c_size_t()
    ctx.check(lib().revnet_transition_workspace_bytes(ctx.h, C.byref(desc), C.byref(f), C.byref(b)), "revnet_transition_workspace_bytes")
    return f.value, b.value


def revnet_transition_fwd(ctx, desc, in1, in2, W, gamma, beta, out1, out2, workspace):
    ctx.check(lib().revnet_transition_fwd(ctx.h, C.byref(desc), _ptr(in1), _ptr(in2), _ptr(W), _ptr(gamma), _ptr(beta),
                                          _ptr(out1), _ptr(out2), _ptr(workspace), _nbytes(workspace), _stream()),
              "revnet_transition_fwd")


def revnet_transition_bwd(ctx, desc, in1, in2, dout1, dout2, W, gamma, beta, din1, din2, dW, dgamma, dbeta, workspace):
    ctx.check(lib().revnet_transition_bwd(ctx.h, C.byref(desc), _ptr(in1), _ptr(in2), _ptr(dout1), _ptr(dout2), _ptr(W),
                                          _ptr(gamma), _ptr(beta), _ptr(din1), _ptr(din2), _ptr(dW), _ptr(dgamma), _ptr(dbeta),
                                          _ptr(workspace), _nbytes(workspace), _stream()), "revnet_transition_bwd")


def revnet_block_fwd_noalloc(ctx, desc, x1, x2, F, G, y1, y2):
    """Block forward on the library's built-in scratch array: for callers that cannot allocate device
    memory.  Same results as revnet_block_fwd; shapes needing more than 16 MiB of scratch are rejected."""
    fp, gp = _fn_params(F), _fn_params(G)
    ctx.check(lib().revnet_block_fwd_noalloc(ctx.h, C.byref(desc), _ptr(x1), _ptr(x2), C.byref(fp), C.byref(gp),
                                             _ptr(y1), _ptr(y2), _stream()), "revnet_block_fwd_noalloc")
