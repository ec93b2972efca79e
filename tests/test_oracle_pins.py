"""The CPU oracle against closed forms, exhaustive enumeration, a hand-worked example,
textbook routines and invariants (no GPU)."""
import pytest

import pins


@pytest.mark.parametrize("order", ["rows", "literal"])
@pytest.mark.parametrize("pin", pins.ALL_PINS, ids=lambda f: f.__name__)
def test_pin(oracle_lib, pin, order):
    if pin in (pins.pin_argmax, pins.pin_literal_equals_rows) and order == "literal":
        pytest.skip("order-independent")
    pin(oracle_lib, order=order)
