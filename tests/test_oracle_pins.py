"""The CPU oracle against what the paper and the mathematics fix (no GPU)."""
import pytest

from tests import oracle_pins


@pytest.mark.parametrize("check", oracle_pins.ALL_CHECKS, ids=lambda f: f.__name__)
def test_pin(oracle, check):
    check(None)          # None -> the committed oracle build
