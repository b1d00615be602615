"""Pins for the oracle's random source: Philox4x32-10 and the draw indexing."""
import os

import numpy as np
import pytest

from oracle import capi, paper_literal as pl
from helpers import GOLDEN


def kat_vectors():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((tuple(w[0:4]), tuple(w[4:6]), tuple(w[6:10])))
    assert len(rows) == 3
    return rows


@pytest.mark.parametrize("ctr,key,expect", kat_vectors())
def test_known_answers(ctr, key, expect):
    assert capi.philox4x32_10(ctr, key) == expect
    assert pl.philox4x32_10(ctr, key) == expect


def test_two_implementations_agree_on_random_counters():
    rng = np.random.default_rng(11)
    for _ in range(200):
        ctr = tuple(int(x) for x in rng.integers(0, 1 << 32, size=4))
        key = tuple(int(x) for x in rng.integers(0, 1 << 32, size=2))
        assert capi.philox4x32_10(ctr, key) == pl.philox4x32_10(ctr, key)


def test_bijection_on_a_small_counter_range():
    # A block cipher in counter mode never repeats an output block under one key.
    outs = {capi.philox4x32_10((c, 0, 0, 0), (5, 6)) for c in range(4096)}
    assert len(outs) == 4096


@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 13, 16])
def test_draw_indexing(k):
    """Draw g is field g mod dpw of word (g mod E)/dpw of block g/E, in both oracles."""
    seed = 0x1234_5678_9ABC_DEF0
    dpw = 32 // k
    E = 4 * dpw
    for g in list(range(0, 3 * E + 5)) + [2 ** 32 * E - 1, 2 ** 32 * E, 2 ** 40 + 17]:
        b = g // E
        out = capi.philox4x32_10((b & 0xFFFFFFFF, b >> 32, 0, 0), (seed & 0xFFFFFFFF, seed >> 32))
        expect = (out[(g % E) // dpw] >> ((g % dpw) * k)) & ((1 << k) - 1)
        assert capi.draw(seed, g, k) == expect
        assert pl.draw(seed, g, k) == expect


@pytest.mark.parametrize("k", [1, 2, 3, 6, 8, 13, 16])
def test_word_stream_matches_draws(k):
    seed, dpw = 99, 32 // k
    offset = 7 * dpw
    count = 9 * 4 * dpw + 3
    words = capi.random_words(seed, offset, count, k)
    for i in range(count):
        assert pl.field_of_words(words, i, k) == capi.draw(seed, offset + i, k)


def test_stream_word_separates_sequences():
    assert capi.draw(1, 0, 8, 0) != capi.draw(1, 0, 8, 1) or capi.draw(1, 1, 8, 0) != capi.draw(1, 1, 8, 1)


@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_draws_are_uniform(k):
    n = 1 << 16
    d = np.array([capi.draw(42, g, k) for g in range(n)])
    counts = np.bincount(d, minlength=1 << k)
    expect = n / (1 << k)
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    dof = (1 << k) - 1
    assert chi2 < dof + 6 * (2 * dof) ** 0.5 + 10
