"""Test-side names for the oracle's level builders."""
from oracle.problems import (  # noqa: F401
    correct_reweight_levels, logreg_levels, quadratic_levels, reweight_levels, three_levels,
)
