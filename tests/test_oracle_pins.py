"""The CPU oracle against what the paper and mathematics fix (no GPU needed)."""
import pytest

from oracle import ref
from tests.oracle_pins import ALL_PINS


@pytest.mark.parametrize("pin", ALL_PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(ref.load())
