"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test names the passage it checks.  References come from tests/exact_ref.py
(sequence-level brute force in 60-digit decimals, counting definitions of the
truncations), from closed forms, or from the small fixtures in tests/golden/.
"""
import math
import os
from decimal import Decimal
from fractions import Fraction

import numpy as np
import pytest

from tests import exact_ref as ex

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F32, BF16 = 0, 1


def _rows(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _golden_kv(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


# --------------------------------------------------------------------------- Example, Sec. 4.2
def test_worked_example_naive_code(orc):
    g = _golden_kv("example_bias.txt")
    logits = _rows([[math.log(g["p_A"]), math.log(g["p_B"])]])
    o = orc.step(logits, F32, np.array([g["code"]]))
    assert o.status[0] == 0 and o.tokens[0] == int(g["token"])
    assert o.codes[0] == pytest.approx(g["rescaled_num"] / g["rescaled_den"], rel=1e-7)
    assert o.p_tok[0] == pytest.approx(g["p_A"], rel=1e-7)


def test_worked_example_shift_removes_bias(orc):
    # Proposition 3 on the example: averaged over the shift, P(token A) = 0.6 with N = 1.
    g = _golden_kv("example_bias.txt")
    logits = _rows([[math.log(g["p_A"]), math.log(g["p_B"])]])
    K = 20000
    us = (np.arange(K) + 0.5) / K
    hits = 0
    for u in us:
        c = orc.lattice_codes(1, float(u))
        hits += int(orc.step(logits, F32, c).tokens[0] == 0)
    assert hits / K == pytest.approx(g["shifted_mean_A"], abs=2.0 / K)


# --------------------------------------------------------------------------- lattice, Def. Sec. 4.2 / Eq. 2
@pytest.mark.parametrize("N", [1, 2, 7, 32, 1000])
def test_lattice_even_on_circle(orc, N):
    for u in [0.0, 0.25, 0.999999, 1.0 - 2 ** -53]:
        c = orc.lattice_codes(N, u)
        assert c.shape == (N,) and (c >= 0).all() and (c < 1).all()
        s = np.sort(c)
        gaps = np.diff(np.concatenate([s, [s[0] + 1.0]]))
        np.testing.assert_allclose(gaps, 1.0 / N, rtol=0, atol=4e-16)
        # the shift of the whole set is u/N
        np.testing.assert_allclose(c[0], u / N, rtol=0, atol=1e-16)


def test_lattice_rejects_bad_arguments(orc):
    for N, u in [(0, 0.5), (-1, 0.5), (4, 1.0), (4, -0.1), (4, float("nan"))]:
        with pytest.raises(ValueError):
            orc.lattice_codes(N, u)


def test_lattice_interval_counts(orc):
    # proofs of the duplicate bounds (Sec. 4.3): an interval of length ell holds
    # floor(N ell) or ceil(N ell) of N evenly spaced shifted points.
    rng = np.random.default_rng(5)
    for _ in range(200):
        N = int(rng.integers(1, 65))
        u = float(rng.random())
        a, ell = float(rng.random()), float(rng.random())
        c = orc.lattice_codes(N, u)
        inside = int((((c - a) % 1.0) < ell).sum())
        assert math.floor(N * ell - 1e-9) <= inside <= math.ceil(N * ell + 1e-9)


def test_appendix_b_constants(orc):
    with open(os.path.join(GOLD, "appendix_b.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for n_s, con_s, coff_s in rows:
        N = int(n_s)
        M = N + 1
        K = 8 * N * M
        e_ll = Fraction(0)
        e_lr = Fraction(0)
        for k in range(K):
            u = (k + 0.5) / K        # midpoints: never on a breakpoint, average is exact
            c = orc.lattice_codes(M, u)
            l = int((c < 1.0 / N).sum())
            r = int(((c >= 1.0 / N) & (c < 2.0 / N)).sum())
            e_ll += Fraction(l * (l - 1), K)
            e_lr += Fraction(l * r, K)
        mu2 = Fraction(M * (M - 1), N * N)
        assert e_ll - mu2 == Fraction(con_s)
        assert e_lr - mu2 == Fraction(coff_s)


# --------------------------------------------------------------------------- one step: interval semantics
def test_step_measure_of_each_token_equals_probability(orc):
    # Sec. 3.1: token i owns an interval of length P(x_i), intervals in vocabulary order.
    rng = np.random.default_rng(11)
    V = 7
    logits = _rows(rng.normal(0, 2, (1, V)))
    p = [float(x) for x in ex.conditional([float(v) for v in logits[0]])]
    M = 40000
    codes = (np.arange(M) + 0.5) / M
    o = orc.step(np.repeat(logits, M, 0), F32, codes)
    assert (o.status == 0).all()
    assert (np.diff(o.tokens) >= 0).all()            # vocabulary order along the code axis
    for j in range(V):
        assert (o.tokens == j).mean() == pytest.approx(p[j], abs=1.5 / M)
    # rescaled code = position inside the interval
    cdf = np.concatenate([[0.0], np.cumsum(p)])
    want = (codes - cdf[o.tokens]) / np.array(p)[o.tokens]
    np.testing.assert_allclose(o.codes, want, rtol=0, atol=1e-9)
    np.testing.assert_allclose(o.cdf_lo, cdf[o.tokens], atol=1e-12)
    np.testing.assert_allclose(o.p_tok, np.array(p)[o.tokens], rtol=1e-12)


def test_step_boundaries_half_open(orc):
    # p = (1/4, 1/4, 1/4, 1/4) exactly: a code on a boundary belongs to the upper interval.
    logits = _rows([[1.5, 1.5, 1.5, 1.5]] * 6)
    codes = np.array([0.0, 0.25, 0.75, np.nextafter(0.25, 0), np.nextafter(0.75, 0), 1.0])
    o = orc.step(logits, F32, codes)
    assert o.tokens.tolist() == [0, 1, 3, 0, 2, 3]
    assert o.codes[0] == 0.0 and o.codes[1] == pytest.approx(0.0, abs=1e-15)
    assert (o.codes < 1.0).all() and (o.codes >= 0.0).all()


def test_step_masked_and_nonfinite(orc):
    ninf = -np.inf
    o = orc.step(_rows([[ninf, 0.0, ninf, 0.0]] * 2), F32, np.array([0.25, 0.75]))
    assert o.tokens.tolist() == [1, 3] and o.n_kept.tolist() == [2, 2]
    bad = orc.step(_rows([[0.0, np.nan], [np.inf, 0.0], [ninf, ninf], [0.0, 0.0], [0.0, 0.0]]),
                   F32, np.array([0.5, 0.5, 0.5, 1.5, np.nan]))
    assert (bad.status == orc.ERR_NUMERIC).all() and (bad.tokens == -1).all()
    assert bad.codes[0] == 0.5 and bad.codes[3] == 1.5


def test_step_bf16_storage_is_widened_exactly(orc):
    from paper_2210_15458_b200 import synth
    rng = np.random.default_rng(3)
    x = rng.normal(0, 3, (5, 33)).astype(np.float32)
    bits = synth.f32_to_bf16_bits(x)
    codes = rng.random(5)
    a = orc.step(bits, BF16, codes, temp=0.7, top_k=4)
    b = orc.step(synth.bf16_bits_to_f32(bits), F32, codes, temp=0.7, top_k=4)
    assert (a.tokens == b.tokens).all() and (a.codes == b.codes).all()


# --------------------------------------------------------------------------- modifiers
@pytest.mark.parametrize("temp", [0.1, 0.7, 1.0, 2.5])
def test_temperature(orc, temp):
    # softmax temperature (Sec. 5.1): p_i proportional to exp(l_i / T); with l = T ln n the
    # distribution is n / sum n exactly.
    n = np.array([1, 2, 3, 4, 10], dtype=np.float64)
    logits = _rows([temp * np.log(n)])
    M = 2000
    codes = (np.arange(M) + 0.5) / M
    o = orc.step(np.repeat(logits, M, 0), F32, codes, temp=temp)
    for j in range(5):
        assert (o.tokens == j).mean() == pytest.approx(n[j] / n.sum(), abs=2.0 / M)


def _check_against_counting_definition(orc, logits_row, temp, top_k, top_p, M=3001):
    p = ex.conditional([float(v) for v in logits_row], temp, top_k, top_p)
    codes = (np.arange(M) + 0.5) / M
    o = orc.step(np.repeat(_rows([logits_row]), M, 0), F32, codes, temp=temp, top_k=top_k, top_p=top_p)
    assert (o.status == 0).all()
    kept = sum(1 for x in p if x > 0)
    assert (o.n_kept == kept).all()
    cdf = [Decimal(0)]
    for x in p:
        cdf.append(cdf[-1] + x)
    for i in range(0, M, 7):
        c = ex.D(codes[i])
        tok = next(j for j in range(len(p)) if cdf[j] <= c < cdf[j + 1])
        d = min(c - cdf[tok], cdf[tok + 1] - c)
        if d > Decimal("1e-12"):
            assert o.tokens[i] == tok
            assert o.codes[i] == pytest.approx(float((c - cdf[tok]) / p[tok]), abs=1e-9)
            assert o.p_tok[i] == pytest.approx(float(p[tok]), rel=1e-12)


def test_top_k_counting_definition_with_ties(orc):
    rng = np.random.default_rng(21)
    for trial in range(30):
        V = int(rng.integers(2, 12))
        row = rng.integers(-3, 4, V).astype(np.float32)      # many ties
        k = int(rng.integers(1, V + 2))
        _check_against_counting_definition(orc, row, float(rng.choice([0.5, 1.0, 2.0])), k, 1.0, M=501)


def test_top_k_special_cases(orc):
    rng = np.random.default_rng(22)
    row = _rows([[1.0, 3.0, 3.0, -2.0, 0.5]])
    codes = rng.random(64)
    rows = np.repeat(row, 64, 0)
    k1 = orc.step(rows, F32, codes, top_k=1)
    assert (k1.tokens == 1).all() and (k1.n_kept == 1).all()      # argmax, lowest index among maxima
    np.testing.assert_allclose(k1.codes, codes, atol=1e-15)        # whole interval -> code unchanged
    assert (k1.tie_topk == 2).all()
    base = orc.step(rows, F32, codes)
    for k in (0, 5, 6, 100):
        kk = orc.step(rows, F32, codes, top_k=k)
        assert (kk.tokens == base.tokens).all() and (kk.codes == base.codes).all()
    k2 = orc.step(rows, F32, codes, top_k=2)                        # the two tied maxima, half each
    assert set(k2.tokens.tolist()) == {1, 2}
    np.testing.assert_allclose(k2.p_tok, 0.5, rtol=1e-15)


def test_nucleus_counting_definition(orc):
    rng = np.random.default_rng(23)
    for trial in range(30):
        V = int(rng.integers(2, 12))
        row = (rng.integers(-4, 5, V) * 0.5).astype(np.float32)
        top_p = float(rng.choice([0.05, 0.3, 0.5, 0.9, 0.99]))
        _check_against_counting_definition(orc, row, float(rng.choice([0.7, 1.0])), 0, top_p, M=501)


def test_nucleus_special_cases(orc):
    rng = np.random.default_rng(24)
    row = _rows([[1.0, 3.0, 3.0, -2.0, 0.5]])
    codes = rng.random(32)
    rows = np.repeat(row, 32, 0)
    tiny = orc.step(rows, F32, codes, top_p=1e-9)
    assert (tiny.tokens == 1).all() and (tiny.n_kept == 1).all()
    base = orc.step(rows, F32, codes)
    for tp in (1.0, 0.0, 1.5, -1.0):
        off = orc.step(rows, F32, codes, top_p=tp)
        assert (off.tokens == base.tokens).all() and (off.codes == base.codes).all()
    # p = (.1, .2, .3, .4): top_p = 0.7 keeps exactly {3, 2}; 0.71 also needs token 1
    row2 = _rows([np.log([1.0, 2.0, 3.0, 4.0])])
    a = orc.step(np.repeat(row2, 32, 0), F32, codes, top_p=0.65)
    b = orc.step(np.repeat(row2, 32, 0), F32, codes, top_p=0.75)
    assert (a.n_kept == 2).all() and set(a.tokens.tolist()) <= {2, 3}
    assert (b.n_kept == 3).all() and set(b.tokens.tolist()) <= {1, 2, 3}
    assert a.d_topp[0] == pytest.approx(0.05, abs=1e-6)


def test_top_k_then_nucleus_order(orc):
    # reading: the nucleus mass is measured on the distribution renormalised over the
    # top-k survivors.  p = (.4,.3,.2,.1); top_k = 2 -> (4/7, 3/7); top_p = .6 then needs both
    # (on the full softmax, .4 + .3 >= .6 as well, but top_p = .5: 4/7 >= .5 keeps ONE token,
    # whereas measured on the full softmax .4 < .5 would keep two).
    row = _rows([np.log([4.0, 3.0, 2.0, 1.0])])
    codes = (np.arange(50) + 0.5) / 50
    o = orc.step(np.repeat(row, 50, 0), F32, codes, top_k=2, top_p=0.5)
    assert (o.n_kept == 1).all() and (o.tokens == 0).all()
    for k, tp in [(3, 0.8), (2, 0.9), (4, 0.35)]:
        _check_against_counting_definition(orc, row[0], 1.0, k, tp, M=301)


# --------------------------------------------------------------------------- whole decode: brute force, Sec. 4.1
def _tiny_model(V, seed, sigma=1.5):
    rng = np.random.default_rng(seed)
    return _rows(rng.normal(0, sigma, (V, V)))


def _book(table, start, T, eos, temp=1.0, top_k=0, top_p=1.0):
    cache = {}

    def row_probs(prev):
        if prev not in cache:
            cache[prev] = ex.conditional([float(v) for v in table[prev]], temp, top_k, top_p)
        return cache[prev]
    return ex.enumerate_codebook(row_probs, start, T, eos)


@pytest.mark.parametrize("V,T,eos,kw", [
    (3, 2, -1, {}),                       # the shape of Fig. 1
    (5, 4, -1, {}),
    (5, 4, 0, {}),                        # EOS makes a prefix-free set of unequal lengths
    (4, 5, 2, {"temp": 0.6}),
    (5, 3, -1, {"top_k": 3}),
    (5, 3, 1, {"top_p": 0.8, "temp": 1.3}),
])
def test_decode_matches_dictionary_order_codebook(orc, V, T, eos, kw):
    table = _tiny_model(V, seed=100 + V * 10 + T)
    start = 1
    book = _book(table, start, T, eos, **kw)
    assert sum(w for _, _, w in book) == pytest.approx(Decimal(1), abs=Decimal("1e-50"))
    rng = np.random.default_rng(7)
    codes = np.concatenate([rng.random(400), (np.arange(100) + 0.5) / 100])
    o = orc.decode_bigram_codes(table, F32, np.full(len(codes), start, np.int32), codes, T, eos, **kw)
    checked = 0
    for i, c in enumerate(codes):
        seq, lo, width, dist = ex.locate(book, c)
        if dist < Decimal("1e-11"):
            continue
        checked += 1
        assert tuple(o.seq[i, :o.len[i]]) == seq
        assert (o.seq[i, o.len[i]:] == -1).all()
        want_final = float((ex.D(c) - lo) / width)
        assert o.codes_final[i] == pytest.approx(want_final, abs=1e-13 / float(width) + 1e-12)
    assert checked > 450


def test_encode_is_the_inverse_map(orc):
    # Sec. 4.1, item (1): sequence -> interval; it must contain the code that produced it.
    table = _tiny_model(6, seed=77)
    rng = np.random.default_rng(8)
    codes = rng.random(200)
    prev = np.full(200, 2, np.int32)
    o = orc.decode_bigram_codes(table, F32, prev, codes, 5, 0, temp=0.8)
    lo, width, st = orc.encode_bigram(table, F32, prev, o.seq, o.len, temp=0.8)
    assert (st == 0).all()
    assert (lo <= codes + 1e-14).all() and (codes < lo + width + 1e-14).all()
    book = _book(table, 2, 5, 0, temp=0.8)
    lut = {seq: (l, w) for seq, l, w in book}
    for i in range(0, 200, 9):
        l, w = lut[tuple(o.seq[i, :o.len[i]])]
        assert lo[i] == pytest.approx(float(l), abs=1e-14)
        assert width[i] == pytest.approx(float(w), rel=1e-13)


def test_lattice_coverage_and_duplicate_bounds(orc):
    # Sec. 4.3 (restated for spacing 1/N): a sequence of probability P is decoded by
    # floor(N P) or ceil(N P) lanes for every shift; in particular P > 1/N => at least once.
    table = _tiny_model(4, seed=55, sigma=2.0)
    T, start, N = 3, 0, 16
    book = _book(table, start, T, -1)
    for u in np.random.default_rng(9).random(25):
        o = orc.decode_bigram(table, F32, np.array([start], np.int32), N, float(u), T, -1)
        got = {}
        for i in range(N):
            got[tuple(o.seq[i])] = got.get(tuple(o.seq[i]), 0) + 1
        for seq, lo, w in book:
            n = got.get(seq, 0)
            assert math.floor(float(w) * N - 1e-9) <= n <= math.ceil(float(w) * N + 1e-9)
            if w > Decimal(1) / N + Decimal("1e-9"):
                assert n >= 1


def test_unbiased_over_shifts_prop3(orc):
    table = _tiny_model(4, seed=56)
    T, start, N = 3, 1, 5
    book = _book(table, start, T, -1)

    def f(seq):
        return 1.0 + 3.0 * seq[0] - 2.0 * seq[-1] + (seq[1] == 2)
    want = float(ex.expectation(book, f))
    K = 4000
    tot = 0.0
    for k in range(K):
        o = orc.decode_bigram(table, F32, np.array([start], np.int32), N, (k + 0.5) / K, T, -1)
        tot += np.mean([f(tuple(s)) for s in o.seq])
    assert tot / K == pytest.approx(want, abs=5e-3)   # deterministic midpoint rule over the shift
    # a biased variant for contrast: the unshifted lattice differs measurably
    o0 = orc.decode_bigram(table, F32, np.array([start], np.int32), N, 0.0, T, -1)
    assert abs(np.mean([f(tuple(s)) for s in o0.seq]) - want) > 5e-3


def test_zero_variance_when_widths_are_multiples_of_1_over_N(orc):
    # Sec. 4.4, first proposition: every sequence of a uniform 4-symbol model with T = 2 has
    # probability exactly 1/16 (token 2 masked out of a 5-symbol vocabulary); with N = 16 each
    # is decoded exactly once for every shift, and with N = 32 exactly twice.
    row = [0.5, 0.5, -np.inf, 0.5, 0.5]
    table = _rows([row] * 5)
    for N in (16, 32):
        for u in np.random.default_rng(10).random(40):
            o = orc.decode_bigram(table, F32, np.array([0], np.int32), N, float(u), 2, -1)
            counts = {}
            for s in o.seq:
                counts[tuple(s)] = counts.get(tuple(s), 0) + 1
            assert len(counts) == 16 and set(counts.values()) == {N // 16}
            assert all(2 not in k for k in counts)


def test_monotone_codes_give_dictionary_ordered_sequences(orc):
    table = _tiny_model(5, seed=57)
    codes = np.sort(np.random.default_rng(12).random(300))
    o = orc.decode_bigram_codes(table, F32, np.full(300, 3, np.int32), codes, 4, -1)
    seqs = [tuple(s) for s in o.seq]
    assert seqs == sorted(seqs)


def test_iid_codes_sample_the_model_prop1(orc):
    table = _tiny_model(3, seed=58)
    book = _book(table, 0, 2, -1)
    n = 60000
    codes = np.random.default_rng(13).random(n)
    o = orc.decode_bigram_codes(table, F32, np.zeros(n, np.int32), codes, 2, -1, threads=4)
    chi2 = 0.0
    for seq, lo, w in book:
        obs = int(((o.seq[:, 0] == seq[0]) & (o.seq[:, 1] == seq[1])).sum())
        chi2 += (obs - n * float(w)) ** 2 / (n * float(w))
    assert chi2 < 30.0           # 8 degrees of freedom; P(chi2 > 30) ~ 2e-4


def test_decode_split_and_resume(orc):
    table = _tiny_model(6, seed=59)
    codes = np.random.default_rng(14).random(50)
    prev = np.full(50, 4, np.int32)
    full = orc.decode_bigram_codes(table, F32, prev, codes, 8, 0)
    a = orc.decode_bigram_codes(table, F32, prev, codes, 4, 0)
    alive = a.len == 4
    alive &= a.seq[:, 3] != 0
    idx = np.nonzero(alive)[0]
    b = orc.decode_bigram_codes(table, F32, a.seq[idx, 3], a.codes_final[idx], 4, 0)
    for n, i in enumerate(idx):
        assert (full.seq[i, 4:] == b.seq[n]).all()
        assert full.codes_final[i] == b.codes_final[n]


def test_threads_do_not_change_results(orc):
    rng = np.random.default_rng(15)
    logits = _rows(rng.normal(0, 2, (37, 50)))
    codes = rng.random(37)
    a = orc.step(logits, F32, codes, temp=0.9, top_k=7, top_p=0.9)
    b = orc.step(logits, F32, codes, temp=0.9, top_k=7, top_p=0.9, threads=5)
    assert (a.tokens == b.tokens).all() and (a.codes == b.codes).all()


# --------------------------------------------------------------------------- n-gram diversity (Sec. 5.1)
def _diversity_by_sets(seq, length, N):
    """The definition with Python sets: distinct n-grams over all n-grams, per group."""
    lanes, T = seq.shape
    out_u, out_t, out_d = [], [], []
    for g in range(lanes // N):
        us, ts, d = [], [], Fraction(0)
        for n in (1, 2, 3, 4):
            grams = [tuple(int(v) for v in seq[i, t:t + n]) for i in range(g * N, (g + 1) * N)
                     for t in range(0, min(int(length[i]), T) - n + 1)]
            us.append(len(set(grams)))
            ts.append(len(grams))
            if grams:
                d += Fraction(len(set(grams)), len(grams))
        out_u.append(us)
        out_t.append(ts)
        out_d.append(float(d))
    return np.array(out_u), np.array(out_t), np.array(out_d)


def test_diversity_hand_example(orc):
    # two sequences (1 2 3) and (1 2 4 5): unigrams 1 2 3 1 2 4 5 -> 5 distinct of 7; bigrams
    # (1 2)(2 3)(1 2)(2 4)(4 5) -> 4 of 5; trigrams (1 2 3)(1 2 4)(2 4 5) -> 3 of 3; one 4-gram
    seq = np.array([[1, 2, 3, -1], [1, 2, 4, 5]], np.int32)
    u, t, d = orc.ngram_diversity(seq, np.array([3, 4], np.int32), 2)
    assert u.tolist() == [[5, 4, 3, 1]] and t.tolist() == [[7, 5, 3, 1]]
    assert d[0] == pytest.approx(5 / 7 + 4 / 5 + 1 + 1, abs=1e-15)


def test_diversity_closed_forms(orc):
    T, N = 9, 6
    # N copies of one sequence of distinct tokens: every n-gram occurs N times -> d_n = 1/N
    same = np.tile(np.arange(10, 10 + T, dtype=np.int32), (N, 1))
    u, t, d = orc.ngram_diversity(same, np.full(N, T, np.int32), N)
    assert u.tolist() == [[T, T - 1, T - 2, T - 3]] and t.tolist() == [[N * T, N * (T - 1), N * (T - 2), N * (T - 3)]]
    assert d[0] == pytest.approx(4.0 / N, abs=1e-15)
    # all tokens distinct across the group: nothing repeats -> d = 4
    distinct = np.arange(N * T, dtype=np.int32).reshape(N, T)
    u, t, d = orc.ngram_diversity(distinct, np.full(N, T, np.int32), N)
    assert (u == t).all() and d[0] == 4.0
    # one repeated token: a single unigram, bigram, ... whatever the length
    ones = np.full((N, T), 7, np.int32)
    u, t, d = orc.ngram_diversity(ones, np.full(N, T, np.int32), N)
    assert u.tolist() == [[1, 1, 1, 1]]
    # lengths below n give no n-grams; an empty group scores 0 (reading: empty ratio = 0)
    short = np.array([[3, 4, -1, -1], [3, -1, -1, -1], [-1, -1, -1, -1]], np.int32)
    u, t, d = orc.ngram_diversity(short, np.array([2, 1, 0], np.int32), 3)
    assert t.tolist() == [[3, 1, 0, 0]] and u.tolist() == [[2, 1, 0, 0]]
    assert d[0] == pytest.approx(2 / 3 + 1.0, abs=1e-15)
    u, t, d = orc.ngram_diversity(short, np.zeros(3, np.int32), 3)
    assert t.sum() == 0 and d[0] == 0.0
    # padding is never part of an n-gram, whatever value it holds
    a = np.array([[5, 6, 7, 8, 9], [5, 6, 1, 1, 1]], np.int32)
    b = a.copy()
    b[1, 2:] = -1
    ua, ta, da = orc.ngram_diversity(a, np.array([5, 2], np.int32), 2)
    ub, tb, db = orc.ngram_diversity(b, np.array([5, 2], np.int32), 2)
    assert (ua == ub).all() and (ta == tb).all() and da[0] == db[0]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_diversity_against_set_counting(orc, seed):
    rng = np.random.default_rng(seed)
    S, N, T = 5, 7, 11
    seq = rng.integers(0, 4 + 3 * seed, (S * N, T)).astype(np.int32)      # small alphabets: many repeats
    length = rng.integers(0, T + 1, S * N).astype(np.int32)
    for i in range(S * N):
        seq[i, length[i]:] = -1
    u, t, d = orc.ngram_diversity(seq, length, N)
    wu, wt, wd = _diversity_by_sets(seq, length, N)
    assert (u == wu).all() and (t == wt).all()
    np.testing.assert_allclose(d, wd, rtol=0, atol=1e-14)


def test_diversity_of_decoded_groups_lattice_vs_iid(orc):
    # Sec. 5.1's observation in miniature: at equal temperature a group decoded from lattice
    # codes is at least as diverse on average as one decoded from iid codes
    table = _tiny_model(12, seed=77, sigma=1.5)
    N, T, S = 8, 6, 40
    starts = np.arange(S, dtype=np.int32) % 12
    rng = np.random.default_rng(5)
    lat = orc.decode_bigram(table, F32, starts, N, 0.37, T, -1)
    iid = orc.decode_bigram_codes(table, F32, np.repeat(starts, N).astype(np.int32), rng.random(S * N), T, -1)
    d_lat = orc.ngram_diversity(lat.seq, lat.len, N)[2].mean()
    d_iid = orc.ngram_diversity(iid.seq, iid.len, N)[2].mean()
    assert d_lat > d_iid


# --------------------------------------------------------------------------- sample-mean estimator (Sec. 4.2)
def test_reward_mean_is_exact_when_widths_are_multiples_of_1_over_N(orc):
    # one step over 4 symbols with probabilities 1/8, 3/8, 2/8, 2/8 (as exactly as fp32 logits
    # allow): N = 8 lattice codes hit the symbols 1, 3, 2, 2 times for every shift that keeps
    # 1e-6 away from the lattice, so the estimator equals the expectation with zero variance
    p = np.array([1, 3, 2, 2]) / 8.0
    table = _rows([np.log(p)] * 4)
    r = np.array([0.25, -1.5, 4.0, 10.0])
    want = float((p * r).sum())
    for u in [0.013, 0.3, 0.5, 0.77, 0.999]:
        o = orc.decode_bigram(table, F32, np.array([0], np.int32), 8, u, 1, -1)
        lane, mean = orc.reward_mean(o.seq, o.len, 8, r)
        assert np.bincount(o.seq[:, 0], minlength=4).tolist() == [1, 3, 2, 2]
        assert mean[0] == pytest.approx(want, abs=1e-14)
        assert lane.tolist() == [r[t] for t in o.seq[:, 0]]


def test_reward_mean_is_unbiased_over_shifts(orc):
    # Sec. 4.2's proposition against the exact expectation from the enumerated codebook
    table = _tiny_model(4, seed=91)
    T, start, N, eos = 4, 2, 3, 0
    book = _book(table, start, T, eos)
    r = np.array([0.5, -2.0, 3.0, 1.25])
    want = float(ex.expectation(book, lambda seq: sum(r[t] for t in seq)))
    K = 3000
    tot = 0.0
    for k in range(K):
        o = orc.decode_bigram(table, F32, np.array([start], np.int32), N, (k + 0.5) / K, T, eos)
        lane, mean = orc.reward_mean(o.seq, o.len, N, r)
        for i in range(N):                                   # per lane: padding adds nothing
            assert lane[i] == pytest.approx(sum(r[t] for t in o.seq[i, :o.len[i]]), abs=1e-14)
        tot += mean[0]
    assert tot / K == pytest.approx(want, abs=5e-3)


def test_reward_mean_groups_and_bad_tokens(orc):
    seq = np.array([[0, 1, -1], [2, 2, 2], [1, -1, -1], [0, 0, 1]], np.int32)
    ln = np.array([2, 3, 1, 3], np.int32)
    r = np.array([1.0, 10.0, 100.0])
    lane, mean = orc.reward_mean(seq, ln, 2, r)
    assert lane.tolist() == [11.0, 300.0, 10.0, 12.0] and mean.tolist() == [155.5, 11.0]
    with pytest.raises(ValueError):
        orc.reward_mean(np.array([[5]], np.int32), np.array([1], np.int32), 1, r)


# --------------------------------------------------------------------------- the paper's own code sets
def test_lattice_variants_closed_forms(orc):
    for N in (1, 2, 5, 16, 257):
        naive = orc.lattice_codes_variant(N, 0.0, 2)
        assert naive.tolist() == [float(Fraction(i, N + 1)) for i in range(1, N + 1)]
        for b in (0.0, 0.25, 0.999):
            got = orc.lattice_codes_variant(N, b, 1)
            want = [(Fraction(i, N + 1) + Fraction(b)) % 1 for i in range(1, N + 1)]
            assert got == pytest.approx([float(w) for w in want], abs=2e-16)
            assert ((got >= 0) & (got < 1)).all()
            # on the circle: N - 1 gaps of 1/(N+1) and one of 2/(N+1) -- unlike variant 0, whose
            # gaps are all 1/N; this is why the bounds of Sec. 4.3 are stated for variant 0
            srt = np.sort(got)
            gaps = np.diff(np.concatenate([srt, [srt[0] + 1.0]]))
            assert np.sort(gaps)[:-1] == pytest.approx(1.0 / (N + 1), abs=1e-12) or N == 1
            assert gaps.max() == pytest.approx(2.0 / (N + 1), abs=1e-12)
        assert (orc.lattice_codes_variant(N, 0.3, 0) == orc.lattice_codes(N, 0.3)).all()
    with pytest.raises(ValueError):
        orc.lattice_codes_variant(4, 0.5, 3)
    with pytest.raises(ValueError):
        orc.lattice_codes_variant(4, 1.0, 1)


def test_naive_codebook_example_is_biased_but_consistent(orc):
    # the example after the proposition "Naive arithmetic sampling": symbols A (0.6) and B (0.4),
    # N = 1 gives the code 0.5, which always decodes to A: the sample mean of 1[B] is 0, not 0.4
    table = _rows([np.log([0.6, 0.4])] * 2)
    c = orc.lattice_codes_variant(1, 0.0, 2)
    assert c.tolist() == [0.5]
    o = orc.decode_bigram_codes(table, F32, np.array([0], np.int32), c, 1, -1)
    assert o.seq[0, 0] == 0
    # consistency (Eq. of that proposition): the mean over N naive codes tends to E[s] as 1/N
    for N in (10, 100, 1000):
        codes = orc.lattice_codes_variant(N, 0.0, 2)
        o = orc.decode_bigram_codes(table, F32, np.zeros(N, np.int32), codes, 1, -1)
        assert abs((o.seq[:, 0] == 1).mean() - 0.4) <= 1.0 / N


# --------------------------------------------------------------------------- d_tok, the gate of every GPU comparison
def test_d_tok_is_the_distance_to_the_nearest_cdf_boundary_exact(orc):
    # Algorithm 1's interval (m, M) of the chosen token: d_tok = min(c - m, M - c).  With equal
    # logits every kept token has probability 1/n exactly; for n a power of two the CDF values
    # k/n and the codes below are dyadic, so every quantity is exact in fp64 and the oracle must
    # return the distance bit for bit (a division by Z too many, a wrong end, a swapped sign fail).
    ninf = -np.inf
    for row, kept in [([0.5] * 8, list(range(8))),
                      ([1.25, ninf, 1.25, 1.25, ninf, ninf, 1.25, ninf], [0, 2, 3, 6])]:
        n = len(kept)
        codes = (np.arange(256) + 0.25) / 256
        o = orc.step(np.repeat(_rows([row]), len(codes), 0), F32, codes, temp=0.7)
        assert (o.status == 0).all()
        for c, tok, d, lo, p in zip(codes, o.tokens, o.d_tok, o.cdf_lo, o.p_tok):
            i = int(c * n)                                   # position among the kept tokens
            assert tok == kept[i] and p == 1.0 / n and lo == i / n
            assert d == min(c - i / n, (i + 1) / n - c)


def test_d_tok_against_the_decimal_cdf(orc):
    # the same quantity on rows of unequal probabilities, against the CDF in 60-digit decimals,
    # with temperature and both cuts
    rng = np.random.default_rng(91)
    for temp, k, tp in [(1.0, 0, 1.0), (0.6, 4, 1.0), (1.4, 0, 0.8), (0.9, 5, 0.7)]:
        row = _rows([rng.normal(0, 2, 9)])
        p = ex.conditional([float(v) for v in row[0]], temp, k, tp)
        cdf = [Decimal(0)]
        for x in p:
            cdf.append(cdf[-1] + x)
        codes = rng.random(300)
        o = orc.step(np.repeat(row, len(codes), 0), F32, codes, temp=temp, top_k=k, top_p=tp)
        checked = 0
        for c, tok, d in zip(codes, o.tokens, o.d_tok):
            cd = ex.D(c)
            want = [j for j in range(9) if cdf[j] <= cd < cdf[j + 1]][0]
            dist = min(cd - cdf[want], cdf[want + 1] - cd)
            if dist < Decimal("1e-12"):
                continue
            checked += 1
            assert tok == want
            assert d == pytest.approx(float(dist), abs=1e-14)
        assert checked > 290


# --------------------------------------------------------------------------- encode under a cut, Sec. 4.1 with Sec. 5.1's top-k
@pytest.mark.parametrize("kw", [{"top_k": 3}, {"top_p": 0.7, "temp": 1.2}, {"top_k": 4, "top_p": 0.8}])
def test_encode_under_cuts_matches_the_enumerated_codebook(orc, kw):
    # every sequence of the truncated model owns the interval the brute-force codebook gives it;
    # a sequence with a token outside the kept set has probability zero: status NUMERIC, and the
    # interval returned is that of the prefix before the offending token
    V, T, start, eos = 6, 3, 2, 0
    table = _tiny_model(V, seed=123)
    book = _book(table, start, T, eos, **kw)
    assert len(book) < V ** T                                  # the cut really removes sequences
    seqs = np.full((len(book), T), -1, np.int32)
    lens = np.zeros(len(book), np.int32)
    for i, (s, _, _) in enumerate(book):
        seqs[i, :len(s)] = s
        lens[i] = len(s)
    prev = np.full(len(book), start, np.int32)
    lo, width, st = orc.encode_bigram(table, F32, prev, seqs, lens, **kw)
    assert (st == 0).all()
    for i, (_, l, w) in enumerate(book):
        assert lo[i] == pytest.approx(float(l), abs=1e-14)
        assert width[i] == pytest.approx(float(w), rel=1e-13)
    # the intervals tile [0, 1) in dictionary order
    order = np.argsort(lo, kind="stable")
    np.testing.assert_allclose(lo[order][1:], (lo + width)[order][:-1], atol=1e-14)
    assert (lo + width)[order][-1] == pytest.approx(1.0, abs=1e-14)
    # sequences outside the truncated model
    have = {s for s, _, _ in book}
    bad = []
    for a in range(V):
        for b in range(V):
            for c in range(V):
                s = (a, b, c)
                cut = s if eos not in s else s[:s.index(eos) + 1]
                if cut not in have:
                    bad.append(cut + (-1,) * (T - len(cut)))
    bad = np.array(sorted(set(bad)), np.int32)
    assert len(bad) > 0
    blen = np.array([int((r >= 0).sum()) for r in bad], np.int32)
    lo2, w2, st2 = orc.encode_bigram(table, F32, np.full(len(bad), start, np.int32), bad, blen, **kw)
    assert (st2 == orc.ERR_NUMERIC).all()
    pre = {}
    for s, l, w in book:                                       # interval of a prefix = union of its sequences
        for n in range(len(s) + 1):
            a = pre.setdefault(s[:n], [l, Decimal(0)])
            a[1] += w
    for r, l, w in zip(bad, lo2, w2):
        s = tuple(int(x) for x in r if x >= 0)
        n = max(n for n in range(len(s)) if s[:n] in pre)      # longest prefix with positive probability
        assert l == pytest.approx(float(pre[s[:n]][0]), abs=1e-14)
        assert w == pytest.approx(float(pre[s[:n]][1]), rel=1e-12)


# --------------------------------------------------------------------------- typical decoding (named in Sec. 2)
def test_typical_counting_definition(orc):
    # the locally typical set against its counting definition in 60-digit decimals, with
    # temperature, a preceding top-k, ties between equal logits (lower index first) and masked tokens
    rng = np.random.default_rng(321)
    rows = [rng.normal(0, 2, 12), np.round(rng.normal(0, 1.5, 14)), rng.normal(0, 3, 9)]
    rows[2][4] = -np.inf
    checked = 0
    for row in rows:
        row = _rows([row])
        for temp, k, tp in [(1.0, 0, 0.9), (0.7, 0, 0.5), (1.3, 6, 0.8), (1.0, 0, 0.2), (0.9, 3, 0.95)]:
            p = ex.conditional([float(v) for v in row[0]], temp, k, 1.0, tp)
            V = len(p)
            cdf = [Decimal(0)]
            for x in p:
                cdf.append(cdf[-1] + x)
            codes = (np.arange(200) + 0.5) / 200
            o = orc.step(np.repeat(row, len(codes), 0), F32, codes, temp=temp, top_k=k, typical_p=tp)
            if o.d_topp[0] < 1e-9:
                continue                                   # the cut itself hangs on rounding
            assert o.n_kept[0] == sum(1 for x in p if x > 0)
            for c, tok, pt, d in zip(codes, o.tokens, o.p_tok, o.d_tok):
                cd = ex.D(c)
                want = [j for j in range(V) if cdf[j] <= cd < cdf[j + 1]][0]
                if min(cd - cdf[want], cdf[want + 1] - cd) < Decimal("1e-12"):
                    continue
                checked += 1
                assert tok == want and pt == pytest.approx(float(p[want]), rel=1e-12)
    assert checked > 2000


def test_typical_special_cases(orc):
    # a uniform row: every token is equally typical, the lowest indices fill the mass;
    # typical_p >= 1 keeps everything; a two-point row keeps the token nearer the entropy
    flat = _rows([[0.0] * 10])
    o = orc.step(np.repeat(flat, 50, 0), F32, (np.arange(50) + 0.5) / 50, typical_p=0.35)
    assert (o.n_kept == 4).all() and (o.tokens <= 3).all()
    o = orc.step(np.repeat(flat, 50, 0), F32, (np.arange(50) + 0.5) / 50, typical_p=1.0)
    assert (o.n_kept == 10).all()
    # p = (0.9, 0.1): H = 0.325; -ln p = (0.105, 2.303): token 0 is the typical one
    two = _rows([np.log([0.9, 0.1])])
    o = orc.step(np.repeat(two, 20, 0), F32, (np.arange(20) + 0.5) / 20, typical_p=0.5)
    assert (o.n_kept == 1).all() and (o.tokens == 0).all()
    # p = (0.6, 0.2, 0.2): H = 0.950; -ln p = (0.511, 1.609, 1.609): distances 0.439, 0.659, 0.659 -> 0, then 1
    three = _rows([np.log([0.6, 0.2, 0.2])])
    o = orc.step(np.repeat(three, 20, 0), F32, (np.arange(20) + 0.5) / 20, typical_p=0.7)
    assert (o.n_kept == 2).all() and set(o.tokens.tolist()) == {0, 1}
    with pytest.raises(ValueError):
        orc.step(flat, F32, np.array([0.5]), top_p=0.5, typical_p=0.5)
