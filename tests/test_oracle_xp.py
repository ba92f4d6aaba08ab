"""Pins of the oracle's extended-precision decode (Algorithm 1 in exact arithmetic).

The reference here is an exact-rational replay written with Python integers and Fractions:
it knows nothing of digit streams, shifted-in bits or 64-bit words.  It keeps the current
interval [L, L + range * 2^-k) as exact numbers, subdivides it by the same rule the oracle
documents (2^32 cells of r = range >> 32 units; token j owns the cells [F_j, F_{j+1}); the last
kept token also takes the units left over) and asks which sub-interval holds the rational code.
"""
from fractions import Fraction

import numpy as np
import pytest

from tests import exact_ref as ex

F32, BF16 = 0, 1
TWO32 = 1 << 32


def _rows(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _code(j, u, N):
    """(j + floor(u 2^53)/2^53)/N as an exact rational."""
    return Fraction(j * (1 << 53) + int(np.floor(u * 2.0 ** 53)), N * (1 << 53))


class ExactBook:
    """Nested subdivision of [0,1) by a bigram model's cell tables, in exact arithmetic."""

    def __init__(self, orc, table, temp=1.0, top_k=0, top_p=1.0):
        self.orc, self.table, self.kw = orc, table, dict(temp=temp, top_k=top_k, top_p=top_p)
        self.cache = {}

    def cells(self, prev):
        if prev not in self.cache:
            self.cache[prev] = [int(x) for x in self.orc.xp_row_cells(self.table[prev], F32, **self.kw)]
        return self.cache[prev]

    @staticmethod
    def child(L, rng, k, lo, hi):
        r = rng >> 32
        L2 = L + Fraction(r * lo, 1 << k)
        rng2 = rng - r * lo if hi == TWO32 else r * (hi - lo)
        while rng2 <= (1 << 62):
            rng2 <<= 1
            k += 1
        return L2, rng2, k

    def decode(self, c, start, T, eos=-1):
        L, rng, k, prev, seq = Fraction(0), 1 << 63, 63, start, []
        for _ in range(T):
            cells = self.cells(prev)
            r = rng >> 32
            off = (c - L) * (1 << k)                       # exact offset in units
            assert 0 <= off < rng
            t = min(int(off // r), TWO32 - 1)
            tok = next(j for j in range(len(cells) - 1) if cells[j + 1] > t)
            L, rng, k = self.child(L, rng, k, cells[tok], cells[tok + 1])
            seq.append(tok)
            prev = tok
            if tok == eos:
                break
        return seq, L, Fraction(rng, 1 << k)

    def interval(self, seq, start):
        L, rng, k, prev = Fraction(0), 1 << 63, 63, start
        for tok in seq:
            cells = self.cells(prev)
            assert cells[tok + 1] > cells[tok]
            L, rng, k = self.child(L, rng, k, cells[tok], cells[tok + 1])
            prev = tok
        return L, Fraction(rng, 1 << k)

    def enumerate(self, start, T):
        out = []

        def rec(prefix, prev, L, rng, k):
            if len(prefix) == T:
                out.append((tuple(prefix), L, Fraction(rng, 1 << k)))
                return
            cells = self.cells(prev)
            for tok in range(len(cells) - 1):
                if cells[tok + 1] > cells[tok]:
                    rec(prefix + [tok], tok, *self.child(L, rng, k, cells[tok], cells[tok + 1]))
        rec([], start, Fraction(0), 1 << 63, 63)
        return out


def _model(V, seed, sigma=1.5):
    return _rows(np.random.default_rng(seed).normal(0, sigma, (V, V)))


def test_digits_of_the_lattice_codes(orc):
    # two equally likely tokens: every step halves the interval, so the decoded tokens ARE the
    # binary digits of the code -- 53 bits from the quotient, the rest from the long division
    table = _rows(np.zeros((2, 2)))
    for N, u in [(1, 0.0), (3, 0.7), (7, 0.123456789), (1000, 1.0 - 2.0 ** -53), (2 ** 31 - 1, 0.5)]:
        js = sorted({0, N // 3, N - 1})
        st = np.concatenate([orc.xp_lattice_state(N, u, j0=j, count=1) for j in js])
        o = orc.xp_decode_bigram(table, F32, np.zeros(len(js), np.int32), st, N, 200, -1)
        for row, j in zip(o.seq, js):
            c = _code(j, u, N)
            want = [int(c * (1 << (t + 1))) & 1 for t in range(200)]
            assert row.tolist() == want
    with pytest.raises(ValueError):
        orc.xp_lattice_state(4, 1.0)


def test_cells_quantise_the_cdf(orc):
    # F(P_j) against the CDF in 60-digit decimals: within one cell (plus fp64 rounding), ends at 2^32,
    # tokens outside the kept set own no cell
    rng = np.random.default_rng(5)
    for temp, k, tp in [(1.0, 0, 1.0), (0.7, 4, 1.0), (1.3, 0, 0.8), (0.9, 6, 0.6)]:
        row = _rows(rng.normal(0, 2, 11))
        row[3] = -np.inf
        p = ex.conditional([float(v) for v in row], temp, k, tp)
        cells = [int(x) for x in orc.xp_row_cells(row, F32, temp, k, tp)]
        assert cells[0] == 0 and cells[-1] == TWO32
        acc = 0
        for j in range(11):
            acc += p[j]
            if p[j] == 0:
                assert cells[j + 1] == cells[j]
            if j < max(i for i in range(11) if p[i] > 0):
                assert abs(float(acc) * TWO32 - cells[j + 1]) <= 1.0 + 1e-5


@pytest.mark.parametrize("V,T,eos,kw", [(4, 60, -1, {}), (3, 40, 0, {"temp": 0.7}), (6, 50, -1, {"top_k": 3}),
                                        (5, 45, -1, {"top_p": 0.8, "temp": 1.2})])
def test_decode_is_exact_far_beyond_fp64(orc, V, T, eos, kw):
    # every lattice code decodes to the sequence whose interval in the exact subdivision holds it,
    # at lengths where a 53-bit code has long run out of digits
    table = _model(V, 900 + V)
    book = ExactBook(orc, table, **kw)
    N, u, start = 48, 0.37, 1
    st = orc.xp_lattice_state(N, u)
    o = orc.xp_decode_bigram(table, F32, np.full(N, start, np.int32), st, N, T, eos, **kw)
    assert (o.status == 0).all()
    fp64 = orc.decode_bigram_codes(table, F32, np.full(N, start, np.int32), orc.lattice_codes(N, u), T, eos, **kw)
    differs = 0
    for j in range(N):
        c = _code(j, u, N)
        seq, L, w = book.decode(c, start, T, eos)
        assert o.seq[j, :o.len[j]].tolist() == seq and (o.seq[j, o.len[j]:] == -1).all()
        assert L <= c < L + w
        differs += int(fp64.seq[j, :fp64.len[j]].tolist() != seq)
    if eos < 0:
        assert differs > N // 2          # the 53-bit code really fails at this length


def test_codebook_tiles_the_unit_interval_and_follows_the_model(orc):
    # V = 3, T = 3 (the shape of the paper's toy figure, one step longer): the exact intervals of all
    # sequences tile [0,1) in dictionary order, and each is the model's probability up to the
    # 2^-32 quantisation of every step
    table = _model(3, 11)
    book = ExactBook(orc, table)
    seqs = book.enumerate(1, 3)
    assert len(seqs) == 27
    assert seqs[0][1] == 0 and all(a[1] + a[2] == b[1] for a, b in zip(seqs, seqs[1:]))
    assert seqs[-1][1] + seqs[-1][2] == 1
    assert [s for s, _, _ in seqs] == sorted(s for s, _, _ in seqs)
    cache = {}

    def probs(prev):
        if prev not in cache:
            cache[prev] = ex.conditional([float(v) for v in table[prev]])
        return cache[prev]
    for s, _, w in seqs:
        P, prev = 1.0, 1
        for tok in s:
            P *= float(probs(prev)[tok])
            prev = tok
        assert float(w) == pytest.approx(P, abs=3 * 2.0 ** -31)


def test_whole_sequence_duplicate_bounds(orc):
    # Sec. 4.3 for whole sequences: a sequence whose interval has width w is decoded by floor(N w)
    # or ceil(N w) of the N lanes, for every shift -- checked in exact integer arithmetic on a
    # peaked model, where some 16-token sequences are wide enough to repeat and others are not
    table = _model(4, 55, sigma=6.0)
    book = ExactBook(orc, table)
    N, T, start = 128, 16, 0
    for u in (0.0, 0.31, 0.999):
        st = orc.xp_lattice_state(N, u)
        o = orc.xp_decode_bigram(table, F32, np.full(N, start, np.int32), st, N, T, -1)
        counts = {}
        for row in o.seq:
            counts[tuple(row)] = counts.get(tuple(row), 0) + 1
        assert len(counts) < N                                   # some sequences do repeat
        for s, d in counts.items():
            _, w = book.interval(list(s), start)
            assert (N * w.numerator) // w.denominator <= d <= -((-N * w.numerator) // w.denominator)
        # and every sequence wider than 1/N is there (coverage), found by walking the codebook greedily
        for s, d in counts.items():
            L, w = book.interval(list(s), start)
            assert any(L <= _code(j, u, N) < L + w for j in range(N))


def test_long_decode_on_a_peaked_model_stays_exact(orc):
    # a c4-shaped table (bf16-like spread, Zipf-like column bias) cut to 64 tokens, 128 steps: the code
    # of every lane still lies inside its sequence's interval, whose width is far below 2^-300
    from paper_2210_15458_b200 import synth
    V = 64
    bias = synth.zipf_bias(V, 41)
    table = _rows(np.random.default_rng(40).normal(0, 2.5, (V, V)) + bias[None, :])
    book = ExactBook(orc, table, temp=0.8)
    N, T, start, u = 32, 128, 5, 0.6180339887
    o = orc.xp_decode_bigram(table, F32, np.full(N, start, np.int32), orc.xp_lattice_state(N, u), N, T, -1, temp=0.8)
    seqs = set()
    for j in range(0, N, 3):
        L, w = book.interval(o.seq[j].tolist(), start)
        assert L <= _code(j, u, N) < L + w
        assert w < Fraction(1, 1 << 100)
        seqs.add(tuple(o.seq[j]))
    assert len(seqs) == len(range(0, N, 3))                      # all distinct at this length


def test_split_and_resume_and_bad_state(orc):
    table = _model(5, 77)
    N, start = 16, 2
    st = orc.xp_lattice_state(N, 0.25)
    prev = np.full(N, start, np.int32)
    whole = orc.xp_decode_bigram(table, F32, prev, st, N, 20, -1)
    a = orc.xp_decode_bigram(table, F32, prev, st, N, 8, -1)
    b = orc.xp_decode_bigram(table, F32, a.seq[:, 7].copy(), a.state, N, 12, -1)
    assert np.array_equal(np.concatenate([a.seq, b.seq], axis=1), whole.seq)
    assert np.array_equal(b.state, whole.state)
    bad = st.copy()
    bad[0, 0] = 5                                               # a range outside (2^62, 2^63]
    o = orc.xp_decode_bigram(table, F32, prev, bad, N, 3, -1)
    assert o.status[0] == orc.ERR_NUMERIC and o.len[0] == 0 and (o.status[1:] == 0).all()
