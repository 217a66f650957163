"""Pins of the oracle's bf16-state rule (the cached prefix output stored rounded to bf16): checked
against torch's own float32 -> bfloat16 conversion, against the nearest-of-two-neighbours definition
with ties to even, and for touching the active tokens' rows only."""
import numpy as np
import torch

from oracle import oracle as orc
from tests.helpers import make_shape


def _torch_bf16(x32):
    return torch.from_numpy(x32).to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)


def test_rounding_agrees_with_torch_on_float32_inputs():
    rng = np.random.default_rng(5)
    x = np.concatenate([
        rng.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** rng.integers(-30, 30, 4000).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 3.3895314e38, 1.1754944e-38, 1e-40, -7e-41, 9.2e-41], np.float32),
    ]).astype(np.float32)
    x = x[np.isfinite(x)]
    want = _torch_bf16(x)
    got = orc.round_bf16(x.astype(np.float64))
    fin = np.isfinite(want)                      # torch rounds the largest float32 binade up to inf; so does the rule
    assert (got[fin] == want[fin]).all()
    assert (np.isinf(got[~fin]) == np.isinf(want[~fin])).all() or (~fin).sum() == 0


def test_ties_go_to_the_even_neighbour_and_results_have_eight_significant_bits():
    # 1 + 2^-8 lies half way between 1 and 1 + 2^-7: even neighbour is 1; 1 + 3 * 2^-8 goes up to 1 + 2^-6
    assert orc.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert orc.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    assert orc.round_bf16(np.array([-(1.0 + 2.0 ** -8 + 2.0 ** -40)]))[0] == -(1.0 + 2.0 ** -7)
    rng = np.random.default_rng(6)
    x = rng.standard_normal(2000) * 2.0 ** rng.integers(-20, 20, 2000)
    r = orc.round_bf16(x)
    m, e = np.frexp(r)
    assert (np.round(m * 256) == m * 256).all()            # eight significant bits
    # nearest: no bf16 value is closer (neighbours of r are r -+ one unit in the last place)
    ulp = np.ldexp(1.0, e - 8)
    assert (np.abs(r - x) <= ulp / 2 + 0).all()


def test_only_the_active_rows_of_the_state_are_rounded():
    sh = make_shape(2, 4, 2, 16, 8, 4, 4)
    rng = np.random.default_rng(7)
    o_p = rng.standard_normal((2, 8, 4, 16))
    before = o_p.copy()
    act = np.zeros((2, 8), np.int32)
    act[0, :2] = (1, 6)
    act[1, :1] = (3,)
    na = np.array([2, 1], np.int32)
    orc.round_state_bf16(sh, o_p, act, na)
    touched = np.zeros((2, 8), bool)
    touched[0, [1, 6]] = True
    touched[1, 3] = True
    assert (o_p[~touched] == before[~touched]).all()
    assert (o_p[touched] == orc.round_bf16(before[touched])).all()
    assert (o_p[touched] != before[touched]).any()
