"""The CPU oracle against closed forms, exhaustive enumeration, a hand-worked example,
textbook routines and invariants (no GPU)."""
import pytest

import pins


@pytest.mark.parametrize("order", ["rows", "definition"])
@pytest.mark.parametrize("pin", pins.ALL_PINS, ids=lambda f: f.__name__)
def test_pin(oracle_lib, pin, order):
    if pin in (pins.pin_argmax, pins.pin_definition_equals_rows) and order == "definition":
        pytest.skip("order-independent")
    pin(oracle_lib, order=order)
