"""Helpers shared by the test modules (no codec arithmetic)."""
import numpy as np

import oracle

f32 = np.float32


def find_power_of_two_step_bound(p: int):
    """An absolute bound whose resolved step is exactly 2^p (search the neighbours of 2^(p-1) * 64/63)."""
    guess = f32(2.0 ** (p - 1) * 64.0 / 63.0)
    cand = guess
    for _ in range(8):
        for c in (cand, np.nextafter(cand, f32(np.inf)), np.nextafter(cand, f32(0))):
            ea, s, r = oracle.resolve(oracle.EB_ABS, float(c))
            if float(s) == 2.0 ** p:
                return float(c), s
        cand = np.nextafter(cand, f32(np.inf))
    raise AssertionError("no bound found")
