"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle timing.

Holds data generators only: grammar text, vocabularies, documents, token streams, logits.
"""
from .build import FULL, NAMES, Workload, build, f32_to_bf16_bits  # noqa: F401
