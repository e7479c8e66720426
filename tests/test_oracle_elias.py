"""Pins for the oracle's recursive Elias code (Definition A.1) -- CPU only."""
import math
import os

import numpy as np

from oracle import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_textbook_codewords():
    rows = [l.split() for l in open(os.path.join(GOLD, "elias_omega_codewords.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) >= 20
    for k, word in rows:
        assert O.elias_string(int(k)) == word, k


def test_encoder_and_decoder_are_inverse():
    # The paper states encoder and decoder separately; the oracle implements both literally.
    ks = list(range(1, 70000)) + [int(x) for x in
                                  np.random.default_rng(1).integers(1, 2 ** 32, 3000)]
    ks += [2 ** j for j in range(1, 32)] + [2 ** j - 1 for j in range(2, 33)]
    for k in ks:
        w = O.elias_string(k)
        assert O.elias_parse(w) == (k, len(w))
        # self-delimiting: trailing garbage is not consumed
        assert O.elias_parse(w + "1011") == (k, len(w))


def test_length_recurrence_and_lemma():
    # |Elias(k)| = 1 for k = 1, else bitlen(k) + |Elias(bitlen(k) - 1)| -- and the lemma's
    # log k + log log k + ... + 1 upper bound with floors replaced by exact group sizes.
    def ln(k):
        return 1 if k == 1 else k.bit_length() + ln(k.bit_length() - 1)
    expect = [1, 3, 6, 7, 11, 12, 13, 14, 16, 17, 18, 19, 20, 21, 22, 23, 28]
    for m in range(1, 18):
        assert len(O.elias_string(1 << (m - 1))) == expect[m - 1]
        assert len(O.elias_string((1 << m) - 1)) == expect[m - 1]
    for k in list(range(1, 5000)) + [2 ** 20, 2 ** 31 + 12345]:
        L = len(O.elias_string(k))
        assert L == ln(k)
        # lemma A.2 (1): sum of iterated logs + 1, each term rounded up, bounds the length
        t, bound = float(k), 1.0
        while t > 1.0:
            t = math.log2(t)
            bound += math.floor(t) + 1 if t > 0 else 0
            if t <= 1.0:
                break
        assert L <= bound + 1e-9


def test_prefix_free():
    words = [O.elias_string(k) for k in range(1, 600)]
    for i, a in enumerate(words):
        for j, b in enumerate(words):
            if i != j:
                assert not b.startswith(a)
