"""Float64 CPU oracle: reversible block, Algorithm 1, and a classification stack.

TEST INFRASTRUCTURE ONLY (see the package docstring).  All tensors are NCHW
numpy float64; convolution weights are [Cout, Cin, kh, kw].

Structures (plain Python, built by the caller):
  layer    = {"name": str, "gamma": [Cin], "beta": [Cin], "W": [Cout,Cin,k,k], "stride": int (default 1)}
  function = list of layers, applied first to last; each layer is conv(relu(bn(.)))   (Section 2.2, Eq. 2)
  block    = (F, G)                                                                     (Section 3.1)
  net      = {"stem": {"name","W","stride","pad"}, "maxpool": bool,
              "stages": [{"trans": layer or None, "down": block or None, "c": int, "units": [block, ...]}],
              "fc": {"name","W":[K,C],"b":[K]}, "eps": float}
  A stage's "down" block is the paper-shaped way into the stage (Table "Architectural details" counts the
  down-sampling layer inside the first unit of a stage): a coupling unit whose F contains a stride-2
  layer and whose skip paths are parameter-free shortcuts; it is not invertible, so its input is kept.
"""
import ctypes
import os

import numpy as np

from . import build as _build

_lib = None
_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int)

# running count of dense multiply-add work issued through the conv primitives (2 flops per MAC)
FLOPS = {"conv": 0}


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        for fn in ("oracle_conv_fwd", "oracle_conv_dgrad", "oracle_conv_wgrad"):
            getattr(_lib, fn).argtypes = [_D, _D, _D] + [ctypes.c_int] * 8
            getattr(_lib, fn).restype = None
        _lib.oracle_maxpool_fwd.argtypes = [_D, _D, _I] + [ctypes.c_int] * 7
        _lib.oracle_maxpool_bwd.argtypes = [_D, _I, _D] + [ctypes.c_int] * 6
    return _lib


def _p(x):
    return x.ctypes.data_as(_D)


def _c(x):
    return np.ascontiguousarray(x, dtype=np.float64)


def _osz(n, k, s, p):
    return (n + 2 * p - k) // s + 1


# --------------------------------------------------------------------------- primitives

def conv_fwd(a, w, stride=1, pad=None):
    """out[n,co,i,j] = sum_{ci,kh,kw} w[co,ci,kh,kw] a[n,ci,i*s+kh-p,j*s+kw-p]  (Eq. 2, Conv_kxk)."""
    a, w = _c(a), _c(w)
    N, Ci, H, W = a.shape
    Co, _, k, _ = w.shape
    p = k // 2 if pad is None else pad
    out = np.empty((N, Co, _osz(H, k, stride, p), _osz(W, k, stride, p)))
    _load().oracle_conv_fwd(_p(a), _p(w), _p(out), N, Ci, H, W, Co, k, stride, p)
    FLOPS["conv"] += 2 * out.size * Ci * k * k
    return out


def conv_dgrad(dout, w, in_hw, stride=1, pad=None):
    """Adjoint of conv_fwd with respect to its input."""
    dout, w = _c(dout), _c(w)
    N, Co = dout.shape[:2]
    _, Ci, k, _ = w.shape
    p = k // 2 if pad is None else pad
    H, W = in_hw
    da = np.empty((N, Ci, H, W))
    _load().oracle_conv_dgrad(_p(dout), _p(w), _p(da), N, Ci, H, W, Co, k, stride, p)
    FLOPS["conv"] += 2 * dout.size * Ci * k * k
    return da


def conv_wgrad(dout, a, k, stride=1, pad=None):
    """Adjoint of conv_fwd with respect to its weights."""
    dout, a = _c(dout), _c(a)
    N, Ci, H, W = a.shape
    Co = dout.shape[1]
    p = k // 2 if pad is None else pad
    dw = np.empty((Co, Ci, k, k))
    _load().oracle_conv_wgrad(_p(dout), _p(a), _p(dw), N, Ci, H, W, Co, k, stride, p)
    FLOPS["conv"] += 2 * dout.size * Ci * k * k
    return dw


def maxpool_fwd(a, k=3, s=2, p=1):
    a = _c(a)
    N, C, H, W = a.shape
    Ho, Wo = _osz(H, k, s, p), _osz(W, k, s, p)
    out = np.empty((N, C, Ho, Wo))
    idx = np.empty((N, C, Ho, Wo), dtype=np.int32)
    _load().oracle_maxpool_fwd(_p(a), _p(out), idx.ctypes.data_as(_I), N, C, H, W, k, s, p)
    return out, idx


def maxpool_bwd(dout, idx, in_hw):
    dout = _c(dout)
    N, C, Ho, Wo = dout.shape
    H, W = in_hw
    da = np.empty((N, C, H, W))
    _load().oracle_maxpool_bwd(_p(dout), idx.ctypes.data_as(_I), _p(da), N, C, H, W, Ho, Wo)
    return da


def bn_relu_fwd(t, gamma, beta, eps):
    """a(x) = ReLU(BN(x)) with train-mode batch statistics (Eq. 2): per channel over (n,h,w),
    biased variance.  Returns a and what the backward needs."""
    mu = t.mean(axis=(0, 2, 3), keepdims=True)
    var = ((t - mu) ** 2).mean(axis=(0, 2, 3), keepdims=True)
    r = 1.0 / np.sqrt(var + eps)
    xhat = (t - mu) * r
    b = gamma.reshape(1, -1, 1, 1) * xhat + beta.reshape(1, -1, 1, 1)
    a = np.maximum(b, 0.0)
    return a, (xhat, r, b > 0.0, gamma)


def bn_relu_bwd(da, cache):
    """Backprop through ReLU then train-mode BN, differentiating through the batch mean and variance.
    ReLU'(0) = 0."""
    xhat, r, mask, gamma = cache
    M = xhat.shape[0] * xhat.shape[2] * xhat.shape[3]
    db = da * mask
    dbeta = db.sum(axis=(0, 2, 3))
    dgamma = (db * xhat).sum(axis=(0, 2, 3))
    g = gamma.reshape(1, -1, 1, 1)
    dt = (g * r / M) * (M * db - dbeta.reshape(1, -1, 1, 1) - xhat * dgamma.reshape(1, -1, 1, 1))
    return dt, dgamma, dbeta


# --------------------------------------------------------------------------- storage formats
# The definitions above are exact real arithmetic in float64.  Two OPTIONAL storage roundings
# can be switched on so that the discrete decisions of a low-precision implementation (which
# side of zero a ReLU input falls on, which grid point a stored value rounds to) are taken at
# that implementation's precision rather than at float64's:
#   num["bf16_operands"]: convolution operands (activated input, weights, upstream gradient) are
#       rounded to bfloat16 (8-bit exponent, 7-bit mantissa, round to nearest even) before each
#       convolution; products and sums stay float64.
#   num["frac_bits"] = k > 0: the coupling state is kept on the grid 2^-k: y = x + rint(F 2^k)/2^k,
#       the fixed-point remedy of Section 3.2 ("Numerical error"); reconstruction is then exact.
# With num = None (the default everywhere) nothing is rounded.

def round_bf16(x):
    """Round float64 values to the nearest bfloat16 (ties to even), returned as float64."""
    x = np.asarray(x, np.float64)
    m, e = np.frexp(x)                                      # x = m * 2^e, 0.5 <= |m| < 1
    r = np.rint(m * 256.0) / 256.0                          # 8 significant bits; rint = ties to even
    out = np.ldexp(r, e)
    return np.where(np.isfinite(x), out, x)


def _rb(x, num):
    return round_bf16(x) if num and num.get("bf16_operands") else x


def quantize_state(v, num):
    """Residual-function value as it is added to a fixed-point coupling state."""
    k = num.get("frac_bits", 0) if num else 0
    return np.rint(v * float(1 << k)) / float(1 << k) if k else v


# --------------------------------------------------------------------------- residual functions

def fn_fwd(u, layers, eps, num=None):
    """Residual function: chain of c_k(x) = Conv(ReLU(BN(x))) layers (Eq. 2: Basic = c3(c3(x)),
    Bottleneck = c1(c3(c1(x)))).  Returns the value and per-layer caches."""
    caches = []
    t = u
    for L in layers:
        a, bn = bn_relu_fwd(t, np.asarray(L["gamma"], np.float64), np.asarray(L["beta"], np.float64), eps)
        a = _rb(a, num)
        w = _rb(np.asarray(L["W"], np.float64), num)
        s = L.get("stride", 1)
        caches.append((bn, a, w, s, t.shape[2:], L["name"]))
        t = conv_fwd(a, w, stride=s)
    return t, caches


def fn_bwd(g, caches, grads, num=None):
    """Ordinary backprop (Eq. 1) through a residual function; parameter gradients go into `grads`."""
    for bn, a, w, s, in_hw, name in reversed(caches):
        g = _rb(g, num)
        grads[name + ".W"] = conv_wgrad(g, a, w.shape[2], stride=s)
        da = conv_dgrad(g, w, in_hw, stride=s)
        g, dgamma, dbeta = bn_relu_bwd(da, bn)
        grads[name + ".gamma"] = dgamma
        grads[name + ".beta"] = dbeta
    return g


# --------------------------------------------------------------------------- reversible block

def block_fwd(x1, x2, F, G, eps, keep=False, num=None):
    """y1 = x1 + F(x2); y2 = x2 + G(y1)   (Section 3.1)."""
    f, cF = fn_fwd(x2, F, eps, num)
    y1 = x1 + quantize_state(f, num)
    g, cG = fn_fwd(y1, G, eps, num)
    y2 = x2 + quantize_state(g, num)
    return (y1, y2, (cF, cG)) if keep else (y1, y2)


def block_inverse(y1, y2, F, G, eps, num=None):
    """x2 = y2 - G(y1); x1 = y1 - F(x2)   (Section 3.1)."""
    x2 = y2 - quantize_state(fn_fwd(y1, G, eps, num)[0], num)
    x1 = y1 - quantize_state(fn_fwd(x2, F, eps, num)[0], num)
    return x1, x2


def block_bwd_stored(dy1, dy2, caches, grads, num=None):
    """Ordinary backprop through the forward graph with z1 as an explicit node (Eq. 8), using
    activations kept from the forward pass."""
    cF, cG = caches
    dz1 = dy1 + fn_bwd(dy2, cG, grads, num)
    dx2 = dy2 + fn_bwd(dz1, cF, grads, num)
    dx1 = dz1
    return dx1, dx2


def block_bwd_reconstruct(y1, y2, dy1, dy2, F, G, eps, grads, num=None):
    """Algorithm 1 (BlockReverse): rebuild the inputs from the outputs, then backprop.
    Batch statistics are recomputed from the reconstructed tensors; nothing is kept per block.
    The activations computed while reconstructing are reused for the gradient steps (the 4N form,
    Section 5 "Implementation")."""
    z1 = y1
    gz, cG = fn_fwd(z1, G, eps, num)
    x2 = y2 - quantize_state(gz, num)
    fx, cF = fn_fwd(x2, F, eps, num)
    x1 = z1 - quantize_state(fx, num)
    dz1 = dy1 + fn_bwd(dy2, cG, grads, num)
    dx2 = dy2 + fn_bwd(dz1, cF, grads, num)
    dx1 = dz1
    return x1, x2, dx1, dx2


# --------------------------------------------------------------------------- down-sampling unit (not reversible)
# Section 3.1: a reversible block needs stride 1 (anything else discards information); Section 3.2: such layers keep
# their inputs.  The paper's table counts the down-sampling inside the first unit of a stage without describing it.
# Reading used here: the same coupling with a parameter-free shortcut S on both skip paths,
#     y1 = S(x1) + F(x2),   y2 = S(x2) + G(y1),
# S = 2x2 average pooling with stride 2, then zero channels appended up to the new width; F has one stride-2 layer
# (its first 3x3 for a basic function, the 3x3 in the middle of a bottleneck), G is an ordinary stride-1 function.

def shortcut_fwd(x, c_out):
    N, C, H, W = x.shape
    p = x.reshape(N, C, H // 2, 2, W // 2, 2).mean(axis=(3, 5))
    out = np.zeros((N, c_out, H // 2, W // 2))
    out[:, :C] = p
    return out


def shortcut_bwd(d, c_in):
    """Adjoint of shortcut_fwd: the first c_in channels, each value spread over its 2x2 window with weight 1/4."""
    return np.repeat(np.repeat(d[:, :c_in], 2, axis=2), 2, axis=3) / 4.0


def down_fwd(x1, x2, F, G, eps, num=None):
    c_out = np.asarray(G[0]["W"]).shape[1]
    f, cF = fn_fwd(x2, F, eps, num)
    y1 = quantize_state(shortcut_fwd(x1, c_out), num) + quantize_state(f, num)
    g, cG = fn_fwd(y1, G, eps, num)
    y2 = quantize_state(shortcut_fwd(x2, c_out), num) + quantize_state(g, num)
    return y1, y2, (cF, cG)


def down_bwd(dy1, dy2, caches, c_in, grads, num=None):
    """Ordinary backprop (Eq. 1) through the unit above from its kept input."""
    cF, cG = caches
    dz1 = dy1 + fn_bwd(dy2, cG, grads, num)
    dx2 = shortcut_bwd(dy2, c_in) + fn_bwd(dz1, cF, grads, num)
    dx1 = shortcut_bwd(dz1, c_in)
    return dx1, dx2


# --------------------------------------------------------------------------- classification stack

def softmax_ce(logits, labels):
    """Mean softmax cross-entropy with max-subtracted log-sum-exp; returns loss and dlogits."""
    N = logits.shape[0]
    m = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - m)
    lse = m[:, 0] + np.log(e.sum(axis=1))
    loss = float((lse - logits[np.arange(N), labels]).mean())
    sm = e / e.sum(axis=1, keepdims=True)
    sm[np.arange(N), labels] -= 1.0
    return loss, sm / N


def stack_train_grads(net, images, labels, mode, num=None, keep_blocks=(), keep_transitions=False):
    """Forward + backward of the whole stack.

    mode "stored": every block's activations are kept (ordinary backprop).
    mode "reconstruct": only the inputs of non-reversible layers (stem, max-pool, transitions,
    head) are kept; each stage is reversed block by block with Algorithm 1 (Section 3.2).

    Returns a dict: logits, loss, pred, grads{name: array}, stored_bytes (activation bytes kept
    between forward and backward), block_inputs (the (x1,x2) each block saw in the forward) and,
    in reconstruct mode, recovered (the (x1,x2) Algorithm 1 rebuilt), both keyed (stage, unit).
    For every (stage, unit) in keep_blocks the dict `blocks` also holds what Algorithm 1 was given
    and what it returned there: y1, y2, dy1, dy2, dx1, dx2 (the problem statement of Section 3.2 for
    that block inside the network; reconstruct mode only).  With keep_transitions, `transitions[stage]` holds the stored
    layer's input, its upstream gradient and the gradient it passed on (x, dy, dx).
    """
    eps = net["eps"]
    images = np.asarray(images, np.float64)
    labels = np.asarray(labels).astype(np.int64)
    grads, stored, block_inputs, recovered = {}, [], {}, {}
    blocks, transitions = {}, {}
    assert not keep_blocks or mode == "reconstruct"

    # ---- forward
    st = net["stem"]
    wst = np.asarray(st["W"], np.float64)
    stored.append(images)
    h = conv_fwd(images, wst, stride=st["stride"], pad=st["pad"])
    stem_out_hw = h.shape[2:]
    pool_idx = None
    if net["maxpool"]:
        stored.append(h)                      # nothing of h is needed later except its shape/argmax
        h, pool_idx = maxpool_fwd(h, 3, 2, 1)
    stage_fw = []
    for si, S in enumerate(net["stages"]):
        tcache = None
        if S["trans"] is not None:
            stored.append(h)                  # input of a non-reversible layer is kept
            if keep_transitions:
                transitions[si] = dict(x=h)
            h, tcache = fn_fwd(h, [S["trans"]], eps, num)
        c = S["c"]
        dcache = None
        if S.get("down") is not None:
            stored.append(h)                  # not invertible: its input is kept
            cp = h.shape[1] // 2
            dF, dG = S["down"]
            d1, d2, dcache = down_fwd(h[:, :cp], h[:, cp:], dF, dG, eps, num)
            h = np.concatenate([d1, d2], axis=1)
            dcache = (dcache, cp)
        if si == 0 or S["trans"] is not None:
            h = quantize_state(h, num)        # the stage buffers hold the coupling state's format
        x1, x2 = h[:, :c].copy(), h[:, c:].copy()
        bcaches = []
        for ui, (F, G) in enumerate(S["units"]):
            block_inputs[(si, ui)] = (x1, x2)
            if mode == "stored":
                x1, x2, bc = block_fwd(x1, x2, F, G, eps, keep=True, num=num)
                bcaches.append(bc)
                stored += [t for fc in bc for (bn, a, *_r) in fc for t in (bn[0], a)]
            else:
                x1, x2 = block_fwd(x1, x2, F, G, eps, num=num)
        h = np.concatenate([x1, x2], axis=1)
        stage_fw.append((tcache, bcaches, x1, x2, dcache))
    stored.append(h)                          # top activations: needed to start the reversal
    feat = h.mean(axis=(2, 3))
    fc = net["fc"]
    wfc, bfc = np.asarray(fc["W"], np.float64), np.asarray(fc["b"], np.float64)
    logits = feat @ wfc.T + bfc
    loss, dlogits = softmax_ce(logits, labels)
    pred = logits.argmax(axis=1).astype(np.int32)

    # ---- backward
    grads[fc["name"] + ".W"] = dlogits.T @ feat
    grads[fc["name"] + ".b"] = dlogits.sum(axis=0)
    dfeat = dlogits @ wfc
    Hh, Wh = h.shape[2:]
    dh = np.broadcast_to(dfeat[:, :, None, None] / (Hh * Wh), h.shape).copy()
    for si in reversed(range(len(net["stages"]))):
        S = net["stages"][si]
        tcache, bcaches, y1, y2, dcache = stage_fw[si]
        c = S["c"]
        d1, d2 = dh[:, :c].copy(), dh[:, c:].copy()
        for ui in reversed(range(len(S["units"]))):
            F, G = S["units"][ui]
            rec = dict(y1=y1, y2=y2, dy1=d1, dy2=d2) if (si, ui) in keep_blocks else None
            if mode == "stored":
                d1, d2 = block_bwd_stored(d1, d2, bcaches[ui], grads, num)
            else:
                y1, y2, d1, d2 = block_bwd_reconstruct(y1, y2, d1, d2, F, G, eps, grads, num)
                recovered[(si, ui)] = (y1, y2)
            if rec is not None:
                rec.update(dx1=d1, dx2=d2)
                blocks[(si, ui)] = rec
        if dcache is not None:
            d1, d2 = down_bwd(d1, d2, dcache[0], dcache[1], grads, num)
        dh = np.concatenate([d1, d2], axis=1)
        if tcache is not None:
            if keep_transitions:
                transitions[si]["dy"] = dh
            dh = fn_bwd(dh, tcache, grads, num)
            if keep_transitions:
                transitions[si]["dx"] = dh
    if pool_idx is not None:
        dh = maxpool_bwd(dh, pool_idx, stem_out_hw)
    grads[st["name"] + ".W"] = conv_wgrad(dh, images, wst.shape[2], stride=st["stride"], pad=st["pad"])

    seen, nbytes = set(), 0
    for t in stored:
        if id(t) not in seen:
            seen.add(id(t))
            nbytes += t.size * 4              # counted at the 4-byte storage width of the method
    return dict(logits=logits, loss=loss, pred=pred, grads=grads, stored_bytes=nbytes,
                block_inputs=block_inputs, recovered=recovered, top=(stage_fw[-1][2], stage_fw[-1][3]),
                blocks=blocks, transitions=transitions)


def sgd_step(params, grads, velocity, lr, momentum, weight_decay, decayed):
    """v <- mu v + (g + lambda w) ; w <- w - lr v   (Appendix 6.1: momentum 0.9, weight decay on
    weights named in `decayed` only)."""
    new_p, new_v = {}, {}
    for k, w in params.items():
        w = np.asarray(w, np.float64)
        g = grads[k] + (weight_decay * w if k in decayed else 0.0)
        v = momentum * np.asarray(velocity[k], np.float64) + g
        new_v[k] = v
        new_p[k] = w - lr * v
    return new_p, new_v
