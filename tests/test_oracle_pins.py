"""The CPU oracle against what the paper and mathematics fix (no GPU)."""
import pytest

from oracle import novak_oracle as O
from oracle_pins import ALL_PINS


@pytest.fixture(scope="module")
def lib():
    return O.default_library()


@pytest.mark.parametrize("pin", ALL_PINS, ids=lambda f: f.__name__)
def test_pin(pin, lib):
    pin(lib)
