"""Pins for the oracle's optional storage roundings (`num=`): bfloat16 operand rounding and the
fixed-point coupling state of Section 3.2 ("Numerical error").

Every comparison of the bf16 tensor-core mode runs through these helpers, so each is pinned to
something outside the oracle: the bfloat16 format's own definition (1 sign, 8 exponent, 7 stored
mantissa bits, round to nearest, ties to even — checked by integer arithmetic on the float32 bit
pattern and by torch's CPU conversion), hand-written ties, and the properties Section 3.2 states
(a fixed-point state reconstructs exactly; Algorithm 1 still equals ordinary backprop).  A 7-bit
significand, truncation, ties away from zero or a scale on the wrong side of the rounding fails
at least one test below.
"""
import numpy as np
import pytest
import torch

from oracle import revnet as orc
from paper_1707_04585_b200 import synthetic as syn
from tests import helpers as hp


def bf16_by_bits(x32):
    """bfloat16 rounding of float32 values done on the bit pattern: keep the upper 16 bits, round
    to nearest with ties to the even upper half.  Independent of frexp/rint arithmetic."""
    u = np.asarray(x32, np.float32).view(np.uint32).astype(np.uint64)
    lower = u & 0xFFFF
    upper = u >> 16
    up = (lower > 0x8000) | ((lower == 0x8000) & ((upper & 1) == 1))
    upper = upper + up.astype(np.uint64)
    return (upper << 16).astype(np.uint32).view(np.float32).astype(np.float64)


def bf16_by_integers(x64):
    """Nearest value with an 8-bit significand, ties to even, for float64 input, in exact Python
    integer arithmetic (slow; small arrays only)."""
    out = np.empty(x64.size)
    for i, v in enumerate(np.asarray(x64, np.float64).ravel()):
        if v == 0.0:
            out[i] = v
            continue
        m, e = np.frexp(abs(v))
        n = int(m * (1 << 53))                 # exact: 53-bit significand as an integer
        q, r = divmod(n, 1 << 45)              # keep the top 8 bits
        half = 1 << 44
        if r > half or (r == half and q % 2 == 1):
            q += 1
        out[i] = np.copysign(float(q) * 2.0 ** (e - 8), v)
    return out.reshape(np.shape(x64))


def test_round_bf16_matches_format_definition_over_all_normal_exponents():
    rng = np.random.default_rng(7)
    # every normal float32 exponent short of overflow, random mantissas, both signs
    e = np.repeat(np.arange(-126, 127), 64)
    m = 1.0 + rng.random(e.size)
    x = (np.ldexp(m, e) * rng.choice([-1.0, 1.0], e.size)).astype(np.float32)
    got = orc.round_bf16(x.astype(np.float64))
    assert np.array_equal(got, bf16_by_bits(x))
    assert np.array_equal(got, torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy())
    # float64 inputs that float32 cannot hold: exact integer arithmetic decides
    y = rng.standard_normal(2000) * np.exp(rng.uniform(-30, 30, 2000))
    assert np.array_equal(orc.round_bf16(y), bf16_by_integers(y))
    # 8 significant bits exactly: the result times 2^7 / 2^exponent is an integer, and is within
    # half a unit in the last place of the input
    mant, ex = np.frexp(got)
    assert np.array_equal(mant * 256.0, np.rint(mant * 256.0))
    ulp = np.ldexp(1.0, np.frexp(x.astype(np.float64))[1] - 8)
    assert np.all(np.abs(got - x) <= ulp / 2)


def test_round_bf16_ties_signs_and_fixed_points():
    t = 2.0 ** -8                       # half a unit in the last place for values in [1, 2)
    cases = {
        1.0 + t: 1.0,                   # tie, lower neighbour even
        1.0 + 3 * t: 1.0 + 4 * t,       # tie, upper neighbour even
        1.0 + 5 * t: 1.0 + 4 * t,
        1.0 + 7 * t: 1.0 + 8 * t,
        -(1.0 + t): -1.0,               # sign-symmetric (not round-half-up)
        -(1.0 + 3 * t): -(1.0 + 4 * t),
        1.0 + t + 2.0 ** -30: 1.0 + 2 * t,   # just above a tie goes up (float64 input: no double rounding through float32)
        1.0 + 3 * t - 2.0 ** -30: 1.0 + 2 * t,
        2.0 - t: 2.0,                   # tie that carries into the next exponent
        255.5: 256.0, 254.5: 254.0,     # integers 0..256 are representable; .5 ties to even
        0.0: 0.0, 3.0: 3.0, -0.15625: -0.15625, 2.0 ** -100: 2.0 ** -100, 1.9921875: 1.9921875,
    }
    x = np.array(list(cases))
    want = np.array(list(cases.values()))
    got = orc.round_bf16(x)
    assert np.array_equal(got, want), (x[got != want], got[got != want])
    assert np.signbit(orc.round_bf16(np.array([-0.0])))[0] and not np.signbit(orc.round_bf16(np.array([0.0])))[0]
    # idempotent, odd, and the identity on everything bfloat16 can hold
    rng = np.random.default_rng(8)
    y = rng.standard_normal(4096) * np.exp(rng.uniform(-20, 20, 4096))
    r = orc.round_bf16(y)
    assert np.array_equal(orc.round_bf16(r), r) and np.array_equal(orc.round_bf16(-y), -r)
    every = (np.arange(0x0080, 0x7F80, dtype=np.uint32) << 16).view(np.float32).astype(np.float64)  # all positive normals
    assert np.array_equal(orc.round_bf16(every), every)
    assert np.isnan(orc.round_bf16(np.array([np.nan])))[0] and np.isinf(orc.round_bf16(np.array([np.inf])))[0]


def test_rb_switch_only_rounds_when_asked():
    x = np.array([1.0 + 2.0 ** -12, -3.3])
    assert np.array_equal(orc._rb(x, None), x) and np.array_equal(orc._rb(x, {}), x)
    assert np.array_equal(orc._rb(x, {"frac_bits": 16}), x)
    assert np.array_equal(orc._rb(x, {"bf16_operands": True}), orc.round_bf16(x))


def test_quantize_state_grid_ties_and_identity():
    k = 16
    s = 2.0 ** -k
    num = {"frac_bits": k}
    cases = {
        0.5 * s: 0.0,            # ties to the even grid point
        1.5 * s: 2 * s,
        2.5 * s: 2 * s,
        -0.5 * s: 0.0,
        -1.5 * s: -2 * s,
        0.5 * s + 2.0 ** -40: s,
        1.0: 1.0, -7 * s: -7 * s, 123.456: np.rint(123.456 * 65536) / 65536,
        0.49999 * s: 0.0, 0.50001 * s: s,
    }
    v = np.array(list(cases)); want = np.array(list(cases.values()))
    got = orc.quantize_state(v, num)
    assert np.array_equal(got, want), (v[got != want], got[got != want])
    rng = np.random.default_rng(9)
    x = rng.standard_normal(10000) * 10
    q = orc.quantize_state(x, num)
    assert np.array_equal(q * 65536.0, np.rint(q * 65536.0))          # on the grid 2^-16
    assert np.abs(q - x).max() <= s / 2                                # nearest grid point
    assert np.array_equal(orc.quantize_state(q, num), q)              # idempotent
    assert np.array_equal(orc.quantize_state(-x, num), -q)            # odd: x + q and x - q undo each other
    for k2 in (1, 8, 20):
        q2 = orc.quantize_state(x, {"frac_bits": k2})
        assert np.array_equal(q2 * 2.0 ** k2, np.rint(x * 2.0 ** k2))
    # no grid: the identity (k = 0, missing key, no dict at all)
    for n in (None, {}, {"frac_bits": 0}, {"bf16_operands": True}):
        assert orc.quantize_state(x, n) is x


def _block(kind, seed=5, N=3, H=6, W=5, c=6, w=3):
    b = syn.BlockCfg(N, H, W, c, w, kind, seed=seed)
    inp = syn.make_block_inputs(b, affine_jitter=True)
    F, G = hp.oracle_block(b, inp["params"])
    return b, inp, F, G


NUMS = [{"frac_bits": 16}, {"bf16_operands": True, "frac_bits": 16}, {"frac_bits": 10}]


@pytest.mark.parametrize("kind", ["single", "basic", "bottleneck"])
@pytest.mark.parametrize("num", NUMS)
def test_fixed_point_state_reconstructs_bit_for_bit(kind, num):
    """Section 3.2, "Numerical error": with the coupling state in fixed point the inverse returns
    the inputs exactly, whatever the residual functions compute."""
    b, inp, F, G = _block(kind)
    k = num["frac_bits"]
    x1 = np.rint(inp["x1"].astype(np.float64) * 2.0 ** k) / 2.0 ** k
    x2 = np.rint(inp["x2"].astype(np.float64) * 2.0 ** k) / 2.0 ** k
    y1, y2 = orc.block_fwd(x1, x2, F, G, b.eps, num=num)
    for t in (y1, y2):
        assert np.array_equal(t * 2.0 ** k, np.rint(t * 2.0 ** k))      # outputs stay on the grid
    r1, r2 = orc.block_inverse(y1, y2, F, G, b.eps, num=num)
    assert np.array_equal(r1, x1) and np.array_equal(r2, x2)
    g = {}
    a1, a2, _, _ = orc.block_bwd_reconstruct(y1, y2, inp["dy1"].astype(np.float64), inp["dy2"].astype(np.float64), F, G, b.eps, g, num=num)
    assert np.array_equal(a1, x1) and np.array_equal(a2, x2)
    # the rounding moves the outputs by at most half a grid step per coupling
    p1, p2 = orc.block_fwd(x1, x2, F, G, b.eps)
    if "bf16_operands" not in num:
        assert np.abs(y1 - p1).max() <= 2.0 ** -k / 2 + 1e-12
    # a float state (no grid) does NOT have the property in general: the pin is not vacuous
    f1, f2 = orc.block_fwd(inp["x1"].astype(np.float64), inp["x2"].astype(np.float64), F, G, b.eps)
    q1, q2 = orc.block_inverse(f1, f2, F, G, b.eps)
    assert np.abs(q1 - inp["x1"]).max() <= 1e-12


@pytest.mark.parametrize("kind", ["single", "basic", "bottleneck"])
@pytest.mark.parametrize("num", [{"bf16_operands": True}, {"bf16_operands": True, "frac_bits": 16}, {"frac_bits": 16}])
def test_algorithm1_equals_stored_backprop_with_roundings(kind, num):
    """Algorithm 1 == ordinary backprop stays true under the storage roundings: on a fixed-point
    state both see the same tensors bit for bit; with a float state the recomputed inputs differ
    by rounding only."""
    b, inp, F, G = _block(kind, seed=6)
    k = num.get("frac_bits", 0)
    x1, x2 = inp["x1"].astype(np.float64), inp["x2"].astype(np.float64)
    if k:
        x1, x2 = np.rint(x1 * 2.0 ** k) / 2.0 ** k, np.rint(x2 * 2.0 ** k) / 2.0 ** k
    dy1, dy2 = inp["dy1"].astype(np.float64), inp["dy2"].astype(np.float64)
    y1, y2, caches = orc.block_fwd(x1, x2, F, G, b.eps, keep=True, num=num)
    gs, gr = {}, {}
    s1, s2 = orc.block_bwd_stored(dy1, dy2, caches, gs, num)
    _, _, r1, r2 = orc.block_bwd_reconstruct(y1, y2, dy1, dy2, F, G, b.eps, gr, num=num)
    tol = 0.0 if k else 1e-10
    assert set(gs) == set(gr)
    for a, c in [(s1, r1), (s2, r2)] + [(gs[n], gr[n]) for n in gs]:
        assert hp.rel_l2(c, a) <= tol


def test_bf16_operand_mode_rounds_exactly_the_conv_operands():
    """With bf16_operands the residual function equals the plain one applied to operands that were
    rounded by hand: activated input and weights before each convolution, nothing else."""
    b, inp, F, G = _block("basic", seed=8)
    x = inp["x2"].astype(np.float64)
    num = {"bf16_operands": True}
    got, _ = orc.fn_fwd(x, F, b.eps, num)
    t = x
    for L in F:
        a, _ = orc.bn_relu_fwd(t, np.asarray(L["gamma"], np.float64), np.asarray(L["beta"], np.float64), b.eps)
        t = orc.conv_fwd(bf16_by_integers(a), bf16_by_bits(np.asarray(L["W"], np.float32)))
    assert np.array_equal(got, t)
    plain, _ = orc.fn_fwd(x, F, b.eps)
    e = hp.rel_l2(got, plain)
    assert 1e-4 < e < 2e-2, e            # bf16 has 8 significant bits: the effect is ~2^-9 per operand, not 0 and not 2^-4


def test_num_none_leaves_the_plain_definition_untouched():
    b, inp, F, G = _block("bottleneck", seed=9)
    x1, x2 = inp["x1"].astype(np.float64), inp["x2"].astype(np.float64)
    a = orc.block_fwd(x1, x2, F, G, b.eps)
    for n in (None, {}, {"frac_bits": 0}, {"bf16_operands": False}):
        c = orc.block_fwd(x1, x2, F, G, b.eps, num=n)
        assert np.array_equal(a[0], c[0]) and np.array_equal(a[1], c[1])


def test_stack_on_fixed_point_state_recovers_every_block_input_exactly():
    cfg = hp.tiny_stack("bottleneck", maxpool=True, N=4)
    inp = syn.make_stack_inputs(cfg, affine_jitter=True)
    net = hp.oracle_net(cfg, inp["params"])
    for num in ({"frac_bits": 16}, {"bf16_operands": True, "frac_bits": 16}):
        o = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct", num=num)
        s = orc.stack_train_grads(net, inp["images"], inp["labels"], "stored", num=num)
        for key, (x1, x2) in o["block_inputs"].items():
            r1, r2 = o["recovered"][key]
            assert np.array_equal(r1, x1) and np.array_equal(r2, x2), key
        for k in s["grads"]:
            assert np.array_equal(o["grads"][k], s["grads"][k]), k
