"""Seeded synthetic inputs (corpus, prompts, continuations, weights) shared by the CPU oracle's
tests and the device path's tests and benchmark.  Input data only."""
from . import configs, corpus, rng, weights  # noqa: F401
