"""Seeded synthetic inputs and the traced programs of the benchmark configurations.

This package holds no tensor arithmetic: it draws input arrays from a seeded
generator and states, as a sequence of `op` calls on whatever backend object it
is given, *which* ops each configuration traces.  What an op computes is
defined separately by each backend.
"""
