"""Seeded synthetic-input generators shared by the tests, the benchmark and the oracle pins.

Holds no arithmetic of the verification method itself."""
from . import configs, gen, philox  # noqa: F401
