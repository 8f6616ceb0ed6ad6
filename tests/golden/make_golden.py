"""Writes tests/golden/hash_chains.txt from the CPU oracle alone.

The stored chains are regression values for the oracle's block-chain hashing; the test that
reads them also re-derives each one with an independent XXH64 library when one is importable,
so the file never vouches for itself.  Run:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402

CASES = [
    # name, block_tokens, root_seed, token rule, length
    ("iota48_b16_root0", 16, 0, "iota", 48),
    ("iota41_b16_root0", 16, 0, "iota", 41),
    ("iota48_b16_root1", 16, 1, "iota", 48),
    ("iota96_b32_root0", 32, 0, "iota", 96),
    ("affine64_b16_root0", 16, 0, "affine", 64),
]


def tokens_of(rule, n):
    j = np.arange(n, dtype=np.int64)
    if rule == "iota":
        return j.astype(np.int32)
    return ((1000003 * j + 7) % 128256).astype(np.int32)


def main():
    lines = [
        "# Chained block keys written by tests/golden/make_golden.py from the CPU oracle.",
        "# token rules: iota t_j = j ; affine t_j = (1000003*j + 7) mod 128256",
        "# name block_tokens root_seed rule length : keys (hex)",
    ]
    for name, B, root, rule, n in CASES:
        h, _ = oracle.hash_blocks(tokens_of(rule, n), [0, n], B, root)
        lines.append("%s %d %d %s %d : %s" % (name, B, root, rule, n,
                                              " ".join("%016x" % int(x) for x in h)))
    with open(os.path.join(HERE, "hash_chains.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
