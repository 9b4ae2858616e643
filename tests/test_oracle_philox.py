"""Pins for the oracle's counter-based generator (Philox4x32-10).

The round structure is pinned to numpy's Philox (a 4x64 instance of the same
published construction): a width-generic Python restatement is checked against
numpy at 64 bits, and the oracle's C code against the same restatement at 32
bits.  The four 32-bit constants are checked against the copy in PyTorch's
public header.  Known-answer vectors are deliberately not typed in from memory.
"""
import re
from pathlib import Path

import numpy as np
import pytest

import oracle

CONST = {
    32: dict(M0=0xD2511F53, M1=0xCD9E8D57, W0=0x9E3779B9, W1=0xBB67AE85),
    64: dict(M0=0xD2E7470EE14C6C93, M1=0xCA5A826395121157, W0=0x9E3779B97F4A7C15, W1=0xBB67AE8584CAA73B),
}


def philox4_generic(ctr, key, width, rounds=10):
    """Philox-4xW-R of Salmon, Moraes, Dror, Shaw (SC'11), any word width."""
    mask = (1 << width) - 1
    k = CONST[width]
    c = [int(x) & mask for x in ctr]
    k0, k1 = int(key[0]) & mask, int(key[1]) & mask
    for r in range(rounds):
        if r:
            k0 = (k0 + k["W0"]) & mask
            k1 = (k1 + k["W1"]) & mask
        p0 = k["M0"] * c[0]
        p1 = k["M1"] * c[2]
        c = [(p1 >> width) ^ c[1] ^ k0, p1 & mask, (p0 >> width) ^ c[3] ^ k1, p0 & mask]
    return c


def test_generic_structure_matches_numpy_philox4x64():
    rng = np.random.default_rng(1)
    for _ in range(20):
        ctr = [int(x) for x in rng.integers(0, 2 ** 63, size=4)]
        key = [int(x) for x in rng.integers(0, 2 ** 63, size=2)]
        got = [int(x) for x in np.random.Philox(counter=ctr, key=key).random_raw(4)]
        # numpy advances the counter once before it draws its first block
        bumped = [ctr[0] + 1] + ctr[1:]
        assert got == philox4_generic(bumped, key, 64)


def test_oracle_matches_generic_at_32_bits():
    rng = np.random.default_rng(2)
    cases = [([0, 0, 0, 0], [0, 0]), ([0xFFFFFFFF] * 4, [0xFFFFFFFF] * 2)]
    for _ in range(200):
        cases.append(([int(x) for x in rng.integers(0, 2 ** 32, size=4)],
                      [int(x) for x in rng.integers(0, 2 ** 32, size=2)]))
    for ctr, key in cases:
        assert oracle.philox4x32_10(ctr, key) == philox4_generic(ctr, key, 32)


def test_constants_match_pytorch_public_header():
    import torch
    hdr = Path(torch.__file__).parent / "include" / "ATen" / "core" / "PhiloxRNGEngine.h"
    if not hdr.exists():
        pytest.skip("PyTorch headers not installed")
    text = hdr.read_text().upper()
    for v in CONST[32].values():
        assert f"0X{v:08X}" in text


def test_uniform24_range_and_grid():
    assert oracle.uniform24(0) == 0.0
    assert oracle.uniform24(0xFFFFFFFF) == 1.0 - 2.0 ** -24
    assert oracle.uniform24(0x000000FF) == 0.0          # low 8 bits are dropped
    assert oracle.uniform24(0x80000000) == 0.5


def test_coordinate_to_counter_map():
    seed = (123, 456)
    for i in [0, 1, 2, 3, 4, 5, 127, 128, 1001, 2 ** 34 + 6]:
        for m, t in [(0, 0), (3, 17)]:
            q = i // 4
            block = oracle.philox4x32_10([q & 0xFFFFFFFF, q >> 32, m, t], seed)
            assert oracle.coord_uniform(seed[0], seed[1], i, m, t) == (block[i % 4] >> 8) * 2.0 ** -24


def test_uniformity_chi_square_and_independence_across_streams():
    n, bins = 1 << 16, 64
    u = np.array([oracle.coord_uniform(7, 9, i, 0, 0) for i in range(n)])
    assert u.min() >= 0.0 and u.max() < 1.0
    counts = np.bincount((u * bins).astype(int), minlength=bins)
    chi2 = ((counts - n / bins) ** 2 / (n / bins)).sum()
    assert chi2 < 63 + 6 * np.sqrt(2 * 63)        # mean + 6 sigma of chi2(63)
    # another worker / step / seed gives an unrelated stream
    for other in ([oracle.coord_uniform(7, 9, i, 1, 0) for i in range(4096)],
                  [oracle.coord_uniform(7, 9, i, 0, 1) for i in range(4096)],
                  [oracle.coord_uniform(8, 9, i, 0, 0) for i in range(4096)]):
        r = np.corrcoef(u[:4096], np.array(other))[0, 1]
        assert abs(r) < 6 / np.sqrt(4096)
    # serial correlation of neighbouring coordinates
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 6 / np.sqrt(n)
