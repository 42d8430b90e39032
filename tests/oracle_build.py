"""Test-side names for the oracle's level builders."""
from oracle.problems import logreg_levels, quadratic_levels, reweight_levels, three_levels  # noqa: F401
