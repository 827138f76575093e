"""Parity on seeded random shapes: sizes, dtypes, layouts, epilogues and output types drawn
from a fixed seed, the plan left to choose its own kernel, tile and K split; every result is
compared element by element with the CPU oracle under the acceptance bound."""
import numpy as np
import pytest

import nk_inputs
from nk_testlib import run_and_check

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(20251113764)
    out = []
    for i in range(36):
        dt = "bf16" if i % 3 else "f32"
        layout = "blocked32" if (dt == "bf16" and i % 6 == 1) else "row"
        step = 32 if layout == "blocked32" else (8 if dt == "bf16" else 4)
        M = int(rng.integers(1, 700))
        N = int(rng.integers(1, 160)) * step
        K = int(rng.integers(1, 260)) * step
        if layout == "blocked32":
            M = max(32, M // 32 * 32)
        epi = "bias_relu" if rng.integers(0, 2) else "none"
        out_dt = "bf16" if (dt == "bf16" and rng.integers(0, 2)) else "f32"
        out.append(nk_inputs.Workload(f"rnd{i}_{dt}_{layout}_{M}x{N}x{K}_{epi}_{out_dt}", M, N, K, dt, out_dt,
                                      layout, epi, dist_a=("normal", 1.0), dist_b=("uniform", 1.0),
                                      seed=9000 + i))
    return out


@pytest.mark.parametrize("w", _cases(), ids=lambda w: w.name)
def test_random_shape(w):
    run_and_check(w)
