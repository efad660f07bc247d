"""The learning-rate schedule of the phase driver (host arithmetic only, no GPU)."""
import math

import numpy as np
import pytest

from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import build as libbuild


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return B.load()


def test_bert_schedule_of_the_paper(lib):
    """Section 5.2: linear increase to 4e-4 over the first 12.5K steps, then 0.99 of it after every 520 steps."""
    sc = B.Schedule(23000, 4e-4, 12500, 0.99, 520)
    peak = float(np.float32(4e-4))
    assert B.apms_schedule_lr(sc, 12499) == peak                     # the ramp ends exactly at the peak
    assert B.apms_schedule_lr(sc, 12500) == peak and B.apms_schedule_lr(sc, 12500 + 519) == peak
    assert B.apms_schedule_lr(sc, 0) == float(np.float32(peak / 12500))
    half = B.apms_schedule_lr(sc, 6249)
    assert abs(half - peak / 2) <= 1e-7 * peak
    ramp = [B.apms_schedule_lr(sc, k) for k in range(0, 12500, 97)]
    assert all(b > a for a, b in zip(ramp, ramp[1:]))                # strictly increasing ramp
    d99 = float(np.float32(0.99))
    for j in (1, 2, 10, 100):
        got = B.apms_schedule_lr(sc, 12500 + 520 * j)
        assert got == float(np.float32(peak * d99 ** j))
        assert B.apms_schedule_lr(sc, 12500 + 520 * j - 1) == float(np.float32(peak * d99 ** (j - 1)))
    assert B.apms_schedule_lr(sc, -1) == 0.0


def test_schedule_without_ramp_or_decay(lib):
    flat = B.Schedule(5, 1e-3, 0, 1.0, 0)
    assert {B.apms_schedule_lr(flat, k) for k in (0, 1, 10, 10 ** 9)} == {float(np.float32(1e-3))}
    decay_only = B.Schedule(0, 1.0, 0, 0.5, 3)
    assert [B.apms_schedule_lr(decay_only, k) for k in range(7)] == [1.0, 1.0, 1.0, 0.5, 0.5, 0.5, 0.25]


def test_set_schedule_validates(lib):
    assert lib.apms_set_schedule(None, None) == B.ERR_INVALID_ARG
    assert lib.apms_get_step(None) == -1
