"""The adaptive-KL helper: PPO's published rule around a KL target (host logic only)."""
import math
import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_1912_00167_b200.kl_controller import AdaptiveKL  # noqa: E402


def test_rule_halves_doubles_and_holds():
    c = AdaptiveKL(eta=1.0, kl_target=0.01)
    assert c.update(0.01) == 1.0                      # inside the band
    assert c.update(0.01 / 1.5) == 1.0                # on the lower edge: unchanged
    assert c.update(0.01 / 1.5 - 1e-9) == 0.5         # below: halved
    assert c.update(0.01 * 1.5) == 0.5                # on the upper edge: unchanged
    assert c.update(0.01 * 1.5 + 1e-9) == 1.0         # above: doubled
    assert c.update(float("nan")) == 1.0              # a NaN measurement changes nothing


def test_closed_loop_settles_inside_the_band():
    # a toy policy whose KL after an update is proportional to 1 / eta
    c = AdaptiveKL(eta=100.0, kl_target=0.02)
    kl = None
    for _ in range(60):
        kl = 0.5 / c.eta
        c.update(kl)
    assert 0.02 / 1.5 <= 0.5 / c.eta <= 0.02 * 1.5 * 2.0 and c.eta > 0


def test_bounds_and_bad_arguments():
    c = AdaptiveKL(eta=1e-8, kl_target=1.0)
    assert c.update(0.0) == 1e-8                      # never reaches 0: the library skips the KL term at 0
    c = AdaptiveKL(eta=1e8, kl_target=1.0)
    assert c.update(1e9) == 1e8
    with pytest.raises(ValueError):
        AdaptiveKL(eta=0.0)
    with pytest.raises(ValueError):
        AdaptiveKL(kl_target=-1.0)
    assert math.isfinite(AdaptiveKL().eta)
