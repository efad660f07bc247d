"""The CPU oracle against what the paper and the mathematics fix (no GPU)."""
import pytest

import oracle_pins as pins
from oracle import apms_oracle as ao


@pytest.mark.parametrize("check", pins.ALL_CHECKS, ids=lambda f: f.__name__)
def test_pin(check):
    check(ao.lib())
