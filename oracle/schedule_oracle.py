"""ORACLE -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Approximation schedules (paper Section 2.5): a schedule says, for every
convolution layer and every training batch, whether the filter gradient is
computed in full or replaced by one approximation method.  This module states the
schedules of Section 3 (first schedule, two-layer CNN) and Section 3.4
(schedules 2 and 3) plus the seeded-fraction schedule used by the sweep
workload, as plain Python.  ``approximated(...)`` returns True when layer
``layer`` (0-based) is approximated at training step ``step`` (0-based).

Readings where the paper leaves the phase open (its schedule figures are not
recoverable): "every other batch" means odd steps; "every fourth batch" means
steps with step % 4 == 3; "every other layer" means the 2nd, 4th, ... layer.
"""
from __future__ import annotations

EVERY_4TH_LAYER = 0            # Section 3: every fourth conv layer from the second, every batch
ALT_LAYER_ALT_BATCH = 1        # Section 3.4 schedule 2
ALL_LAYERS_EVERY_4TH_BATCH = 2  # Section 3.4 schedule 3
LAYER2_ALT_BATCH = 3           # Section 3: two-layer CNN, second conv every other batch
SEEDED_FRACTION_ALT_BATCH = 4  # sweep workload: a seeded subset of the layers on odd steps

_MASK64 = (1 << 64) - 1


def splitmix64(x: int) -> int:
    """One output of the SplitMix64 mixer (Steele, Lea, Flood 2014) for state x."""
    z = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def fraction_mask(num_layers: int, fraction: float, seed: int) -> list[bool]:
    """round(fraction*L) layers, chosen as the lowest splitmix64(seed + layer) hashes (ties: lower layer)."""
    m = int(fraction * num_layers + 0.5)
    m = max(0, min(num_layers, m))
    order = sorted(range(num_layers), key=lambda l: (splitmix64((seed + l) & _MASK64), l))
    chosen = set(order[:m])
    return [l in chosen for l in range(num_layers)]


def approximated(kind: int, num_layers: int, layer: int, step: int,
                 fraction: float = 0.0, seed: int = 0) -> bool:
    one_based = layer + 1
    if kind == EVERY_4TH_LAYER:
        return one_based >= 2 and (one_based - 2) % 4 == 0
    if kind == ALT_LAYER_ALT_BATCH:
        return one_based % 2 == 0 and step % 2 == 1
    if kind == ALL_LAYERS_EVERY_4TH_BATCH:
        return step % 4 == 3
    if kind == LAYER2_ALT_BATCH:
        return one_based == 2 and step % 2 == 1
    if kind == SEEDED_FRACTION_ALT_BATCH:
        return step % 2 == 1 and fraction_mask(num_layers, fraction, seed)[layer]
    raise ValueError("unknown schedule kind %r" % (kind,))
