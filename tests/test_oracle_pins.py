"""The committed CPU oracle against its pins (no GPU)."""
import pytest

import oracle
import oracle_pins


@pytest.mark.parametrize("name,pin", oracle_pins.ALL_PINS, ids=[n for n, _ in oracle_pins.ALL_PINS])
def test_pin(name, pin):
    pin(oracle.default())
