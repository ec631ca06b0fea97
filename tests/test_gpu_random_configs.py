"""Randomly drawn small layers through the same parity checks as the hand-picked cases: shapes the tiling rarely meets
(d_ff of 64 or 576, one to 200 experts, capacities from 4 slots up, T that is not a multiple of anything) combined
with randomly chosen options.  The draw is seeded, so the cases are the same on every run; combinations the library
refuses are skipped.  Each case is checked exactly like the named tests: integer state bit for bit, every tensor by
its relative Frobenius error and element by element."""
import random

import pytest

from paper_2101_03961_b200 import inputs as si
from paper_2101_03961_b200 import switch_moe as sm
from tests.gpu_helpers import TOL_BF16, TOL_F32
from tests.test_gpu_parity import _check_layer, _check_top2

pytestmark = pytest.mark.gpu

CASES_PER_SEED = 40


def _draw(rng: random.Random, i: int):
    T = rng.choice([256, 512, 768, 1000, 1536, 2048, 4096])
    d = rng.choice([64, 128, 192, 320])
    f = rng.choice([64, 128, 192, 320, 576])
    E = rng.choice([1, 2, 3, 5, 8, 17, 40, 96, 130, 200])
    cf = rng.choice([0.5, 1.0, 1.25, 2.0, 4.0])
    bias = rng.choice([0.0, 0.3, 1.0])
    kw = {}
    top2 = rng.random() < 0.12 and T % 256 == 0 and E > 1      # (one expert: no second choice, a test of its own)
    if not top2:
        if rng.random() < 0.3:
            kw["residual"] = True
        if rng.random() < 0.35:
            kw["geglu"] = True
        if rng.random() < 0.25:
            kw["dropout"] = 0.3
        if rng.random() < 0.25:
            kw["reroute"] = True
            kw["reroute_stages"] = rng.choice([1, 1, 2, 4])
        elif rng.random() < 0.25 and not kw.get("dropout"):
            groups = rng.choice([2, 4])
            if T % (256 * groups) == 0:
                kw["groups"] = groups
        if rng.random() < 0.2:
            kw["noise_eps"] = 0.3
        if rng.random() < 0.2:
            kw["jitter_eps"] = 0.2
    r = rng.random()
    path = sm.GEMM_SIMT if r < 0.15 else (sm.GEMM_TC_1CTA if r < 0.3 else sm.GEMM_DEFAULT)
    f32 = rng.random() < 0.25                                  # all-float32 layer (its own kernels and tolerance)
    cfg = si.SwitchConfig(f"random{i}", T, d, f, E, cf, bias_std=bias, dtype=si.DTYPE_F32 if f32 else si.DTYPE_BF16)
    capacity = int(T / kw.get("groups", 1) * cf / E)
    return cfg, path, top2, kw, capacity, (TOL_F32 if f32 else TOL_BF16)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_randomly_drawn_layers_match_oracle(seed):
    rng = random.Random(seed)
    checked = 0
    for i in range(CASES_PER_SEED):
        cfg, path, top2, kw, capacity, tol = _draw(rng, i)
        if capacity < 4 or capacity > cfg.T:                   # a handful of tokens per expert: the element-wise bound's
            continue                                           # statistics (many tokens per column) do not hold
        try:
            if top2:
                _check_top2(cfg, path, tol, residual=rng.random() < 0.5, expect_mix=False)
            else:
                _check_layer(cfg, path, tol, d_aux=0.6, **kw)
        except sm.SwitchMoeError:
            continue                                           # a combination the library refuses
        except AssertionError as err:
            raise AssertionError(f"case {i} of seed {seed}: {cfg}, path {path}, top2 {top2}, {kw}") from err
        checked += 1
    assert checked >= CASES_PER_SEED // 3
