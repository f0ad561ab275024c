"""Pins the CPU oracle to the hand-worked windows under tests/golden/."""
import pytest

import golden_checks
from runners import run_oracle


@pytest.mark.parametrize("check", golden_checks.ALL, ids=lambda f: f.__name__)
def test_oracle_matches_hand_worked_window(check):
    check(run_oracle)
