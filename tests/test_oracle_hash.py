"""Pins for the oracle's XXH64 and block-chain keys (CPU only).

The paper prints no hash value, so the pins are: the xxHash project's published self-test
values, an independent XXH64 library (when importable), and invariants of chained keys.
"""
import os
import struct

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1


def _sanity_stream(n):
    g, out = 2654435761, bytearray()
    for _ in range(n):
        out.append((g >> 56) & 0xFF)
        g = (g * 11400714785074694797) & M64
    return bytes(out)


def _published():
    rows = []
    for line in open(os.path.join(GOLDEN, "xxh64_published.txt")):
        if line.startswith("#") or not line.strip():
            continue
        n, seed, hx = line.split()
        rows.append((int(n), int(seed), int(hx, 16)))
    return rows


def test_published_values():
    stream = _sanity_stream(256)
    rows = _published()
    assert len(rows) == 9
    for n, seed, expect in rows:
        assert oracle.xxh64(stream[:n], seed) == expect, (n, seed)


def test_block_sized_vectors():
    """The sizes the path hashes (whole 32-byte stripes, no tail): stored values that the
    independent xxhash library gives for these inputs."""
    n_rows = 0
    for line in open(os.path.join(GOLDEN, "xxh64_block_sized.txt")):
        if line.startswith("#") or not line.strip():
            continue
        what, seed, hx = line.split()
        kind, n = what.split(":")
        data = bytes(int(n)) if kind == "zeros" else bytes(range(int(n)))
        assert oracle.xxh64(data, int(seed)) == int(hx, 16), what
        n_rows += 1
    assert n_rows == 3


def test_against_independent_library():
    xxhash = pytest.importorskip("xxhash")
    rng = np.random.default_rng(7)
    for n in list(range(0, 100)) + [127, 128, 129, 255, 256, 1000, 4096]:
        data = rng.integers(0, 256, n, dtype=np.uint8).tobytes()
        seed = int(rng.integers(0, 1 << 63)) * 2 + int(rng.integers(0, 2))
        assert oracle.xxh64(data, seed) == xxhash.xxh64_intdigest(data, seed), n


def _chain_with_library(tokens, B, root):
    xxhash = pytest.importorskip("xxhash")
    out, parent = [], root
    for i in range(len(tokens) // B):
        msg = struct.pack("<%di" % B, *[int(t) for t in tokens[i * B:(i + 1) * B]])
        parent = xxhash.xxh64_intdigest(msg, parent)
        out.append(parent)
    return out


def _tokens_of(rule, n):
    j = np.arange(n, dtype=np.int64)
    return j.astype(np.int32) if rule == "iota" else ((1000003 * j + 7) % 128256).astype(np.int32)


def test_stored_chains_match_oracle_and_library():
    n_cases = 0
    for line in open(os.path.join(GOLDEN, "hash_chains.txt")):
        if line.startswith("#") or not line.strip():
            continue
        head, vals = line.split(":")
        name, B, root, rule, n = head.split()
        B, root, n = int(B), int(root), int(n)
        expect = [int(v, 16) for v in vals.split()]
        toks = _tokens_of(rule, n)
        h, blk_off = oracle.hash_blocks(toks, [0, n], B, root)
        assert [int(x) for x in h] == expect, name
        assert blk_off.tolist() == [0, n // B]
        assert _chain_with_library(toks, B, root) == expect, name
        n_cases += 1
    assert n_cases == 5


def test_chain_is_seeded_by_parent_key_library():
    # batch of ragged requests, negative and large token ids included
    rng = np.random.default_rng(3)
    lens = [0, 5, 16, 17, 31, 32, 100, 257]
    toks = rng.integers(-5, 2**31 - 1, sum(lens), dtype=np.int64).astype(np.int32)
    off = np.concatenate([[0], np.cumsum(lens)])
    for B in (4, 16, 32):
        for root in (0, 1, M64):
            h, bo = oracle.hash_blocks(toks, off, B, root)
            assert bo[-1] == sum(n // B for n in lens)
            for r, n in enumerate(lens):
                got = [int(x) for x in h[bo[r]:bo[r + 1]]]
                assert got == _chain_with_library(toks[off[r]:off[r + 1]], B, root)


def test_suffix_invariance_and_sensitivity():
    rng = np.random.default_rng(11)
    B = 16
    base = rng.integers(0, 32000, 200).astype(np.int32)
    h0, _ = oracle.hash_blocks(base, [0, 200], B, 0)
    assert len(h0) == 12
    for j in (0, 15, 16, 100, 191, 192, 199):
        edited = base.copy()
        edited[j] ^= 1
        h1, _ = oracle.hash_blocks(edited, [0, 200], B, 0)
        k = j // B
        assert np.array_equal(h0[:k], h1[:k])           # blocks before the edit keep their keys
        assert np.all(h0[k:] != h1[k:])                 # every key from the edited block on moves
    # truncating inside a block drops only that partial block
    h2, _ = oracle.hash_blocks(base[:41], [0, 41], B, 0)
    assert np.array_equal(h2, h0[:2])
    # two requests sharing their first 3 blocks share exactly 3 keys
    other = base.copy()
    other[48:] = rng.integers(0, 32000, 152).astype(np.int32)
    both = np.concatenate([base, other])
    h, bo = oracle.hash_blocks(both, [0, 200, 400], B, 0)
    assert np.array_equal(h[bo[0]:bo[0] + 3], h[bo[1]:bo[1] + 3])
    assert h[bo[0] + 3] != h[bo[1] + 3]


def test_short_and_empty_requests():
    h, bo = oracle.hash_blocks(np.arange(15, dtype=np.int32), [0, 15], 16, 0)
    assert len(h) == 0 and bo.tolist() == [0, 0]
    h, bo = oracle.hash_blocks(np.zeros(0, dtype=np.int32), [0], 16, 0)
    assert len(h) == 0
