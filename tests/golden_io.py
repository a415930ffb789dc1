"""Readers for the hand-written fixtures under tests/golden/."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


def e2m1_values():
    """code -> value (float; -0.0 for code 8)."""
    return {int(tok[0], 16): float(tok[1]) for tok in _lines("e2m1_values.txt")}


def direct_cast_blocks():
    """list of dicts: name, bits (uint16[32]), scale, codes (list of int), bytes (list of int)."""
    out, cur = [], None
    for tok in _lines("direct_cast_blocks.txt"):
        if tok[0] == "block":
            cur = {"name": tok[1]}
            out.append(cur)
        elif tok[0] == "in":
            bits = np.zeros(32, np.uint16)
            for i, h in enumerate(tok[1:]):
                bits[i] = int(h, 16)
            cur["bits"] = bits
        elif tok[0] == "scale":
            cur["scale"] = int(tok[1])
        elif tok[0] == "codes":
            cur["codes"] = [int(ch, 16) for ch in tok[1]]
        elif tok[0] == "bytes":
            cur["bytes"] = [int(h, 16) for h in tok[1:]]
    return out


def linear_block_a():
    d = {}
    for tok in _lines("linear_block_A.txt"):
        d[tok[0]] = [float(t) for t in tok[1:]]
    return d
