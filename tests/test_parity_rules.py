"""The parity bookkeeping itself (tests/parity.py), on made-up tensors: what each rule accepts and rejects."""
import numpy as np
import pytest

from tests import parity as par

rng = np.random.default_rng(0)


def tensors(n=10, size=2000):
    return {f"t{i}": rng.standard_normal(size) for i in range(n)}


def test_stated_rule_is_the_default_and_rejects_what_misses_it():
    ref = tensors(2)
    par.check("rules stated ok", {k: v * (1 + 1e-6) for k, v in ref.items()}, ref, 1e-4)
    with pytest.raises(AssertionError):
        par.check("rules stated miss", {k: v * 1.01 for k, v in ref.items()}, ref, 1e-4, lambda: [{k: v * 1.5 for k, v in ref.items()}])
    assert par.RECORDS[-1]["rule"] == "stated"      # a floor function alone changes nothing: the allow-list decides


def test_floor_rule_needs_the_allow_list_and_is_capped():
    ref = tensors(2)
    noise = {k: rng.standard_normal(v.size) for k, v in ref.items()}
    got = {k: v + 0.05 * noise[k] for k, v in ref.items()}
    alt = [{k: v + 0.03 * rng.standard_normal(v.size) for k, v in ref.items()}]           # the oracle moves by 0.03: bound 0.09
    par.check("rules floor ok", got, ref, 1e-3, lambda: alt, ("t*",))
    assert par.RECORDS[-1]["rule"] == "floor" and not par.RECORDS[-1]["met_stated"]
    with pytest.raises(AssertionError):
        par.check("rules floor miss", {k: v + 0.2 * noise[k] for k, v in ref.items()}, ref, 1e-3, lambda: alt, ("t*",))
    with pytest.raises(AssertionError):                                                   # only t0 is on the list: t1 is held to 1e-3
        par.check("rules floor list", got, ref, 1e-3, lambda: alt, ("t0",))


def test_chaotic_rule_still_rejects_zero_wrong_sign_wrong_size_and_uncorrelated():
    ref = tensors(10)
    alt = [{k: 0.2 * v + rng.standard_normal(v.size) for k, v in ref.items()}]            # the oracle against itself: cosine 0.2
    ok = {k: 0.2 * v + rng.standard_normal(v.size) for k, v in ref.items()}
    par.check("rules chaotic ok", ok, ref, 0.05, lambda: alt, ("*",))
    assert par.RECORDS[-1]["rule"] == "chaotic"
    for name, bad in (("zero", {k: 0 * v for k, v in ref.items()}), ("sign", {k: -v for k, v in ok.items()}),
                      ("size", {k: 3 * v for k, v in ok.items()}), ("uncorrelated", {k: rng.standard_normal(v.size) * 1.02 for k, v in ref.items()})):
        with pytest.raises(AssertionError):
            par.check("rules chaotic " + name, bad, ref, 0.05, lambda: alt, ("*",))


def test_block_floor_rule_is_decided_by_size_not_by_outcome():
    small = [(8, 8, 3)]
    assert not par.block_floor_allowed(1, 4, 8, 8, small) and not par.block_floor_allowed(0, 4, 8, 8, small)
    big = [(512, 128, 1), (128, 128, 3), (128, 512, 1)]
    assert par.block_floor_allowed(1, 2, 56, 56, big) and not par.block_floor_allowed(0, 2, 56, 56, big)
    assert par.block_floor_allowed(0, 2, 14, 14, [(2048, 512, 1), (512, 512, 3), (512, 2048, 1)])
