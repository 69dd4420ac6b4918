"""CPU oracle of the two deployment costs the searches trade against accuracy (test infrastructure:
only tests, the smoke check and the benchmark's CPU baseline may import this package).

Section 4, "Compute Latency Estimates": a configuration's latency is the sum, over layers, of
the benchmarked latency of that layer's kernel at the layer's precision.  Table 1: model size is
the weights' storage, parameters times bits / 8, reported in MB of 1e6 bytes.
"""
from typing import Sequence


def size_bytes(layers, bits: Sequence[int]) -> float:
    """Weights-only storage of the configuration in bytes (Table 1, row "Size")."""
    total = 0.0
    for lay, b in zip(layers, bits):
        total += lay.n_out * lay.k_in * int(b) / 8.0
    return total


def latency_ms(table, bs: Sequence[int], bits: Sequence[int]) -> float:
    """Sum over layers of the table entry for (layer, bits[layer]); table[l][i] belongs to width bs[i]."""
    col = {int(b): i for i, b in enumerate(bs)}
    total = 0.0
    for l, b in enumerate(bits):
        total += float(table[l][col[int(b)]])
    return total
