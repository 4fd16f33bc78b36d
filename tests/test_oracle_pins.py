"""The fp64 oracle against what the paper and the mathematics fix (no GPU needed)."""
import pytest

import oracle.mona_oracle as orc
from tests import oracle_pins


@pytest.mark.parametrize("check", oracle_pins.ALL_CHECKS, ids=lambda f: f.__name__)
def test_pin(check):
    check(orc)
