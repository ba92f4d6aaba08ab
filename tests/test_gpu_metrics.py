"""n-gram diversity (Sec. 5.1) and the sample-mean estimator (Sec. 4.2) on the GPU against the
CPU oracle.  Inputs are synthetic token arrays or the oracle's own decodes; the counts must be
bit-exact, the diversity score too (same fp64 expression), the means agree to rounding."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_15458_b200 import binding
    binding.lib()
    return binding


def _tokens(rng, lanes, T, V, zipf=False, min_len=0):
    if zipf:
        p = 1.0 / np.arange(1, V + 1) ** 1.1
        seq = rng.choice(V, size=(lanes, T), p=p / p.sum()).astype(np.int32)
    else:
        seq = rng.integers(0, V, (lanes, T)).astype(np.int32)
    length = rng.integers(min_len, T + 1, lanes).astype(np.int32)
    for i in range(lanes):
        seq[i, length[i]:] = -1
    return seq, length


def _diversity_both(B, orc, seq, length, N):
    u, t, d = B.as_ngram_diversity(torch.from_numpy(seq).cuda(), torch.from_numpy(length).cuda(), N)
    torch.cuda.synchronize()
    wu, wt, wd = orc.ngram_diversity(seq, length, N)
    assert (u.cpu().numpy() == wu).all()
    assert (t.cpu().numpy() == wt).all()
    assert (d.cpu().numpy() == wd).all()             # same fp64 expression on both sides
    return wu, wt, wd


@pytest.mark.parametrize("S,N,T,V", [(1, 1, 1, 3), (3, 2, 5, 2), (7, 5, 9, 4), (40, 8, 17, 11), (5, 32, 128, 50),
                                     (300, 3, 4, 6), (2, 64, 256, 1000), (1, 16, 1024, 7)])
def test_diversity_random_tokens(B, orc, S, N, T, V):
    rng = np.random.default_rng(S * 1000 + N * 10 + T)
    seq, length = _tokens(rng, S * N, T, V)
    _diversity_both(B, orc, seq, length, N)


def test_diversity_c4_shaped_groups(B, orc):
    # 64 groups of 32 sequences of up to 128 tokens over a 32128-token vocabulary with a
    # Zipf-like unigram law, ragged lengths: the shape of the bigram decode's output
    rng = np.random.default_rng(44)
    seq, length = _tokens(rng, 64 * 32, 128, 32128, zipf=True, min_len=20)
    wu, wt, wd = _diversity_both(B, orc, seq, length, 32)
    assert (wu[:, 0] < wt[:, 0]).all() and (wd > 1.0).all()


def test_diversity_degenerate_inputs(B, orc):
    N, T = 6, 9
    same = np.tile(np.arange(10, 10 + T, dtype=np.int32), (N, 1))
    _, _, d = _diversity_both(B, orc, same, np.full(N, T, np.int32), N)
    assert d[0] == pytest.approx(4.0 / N, abs=1e-15)
    ones = np.full((N, T), 7, np.int32)
    _diversity_both(B, orc, ones, np.full(N, T, np.int32), N)
    # empty sequences, lengths above T (clamped), T = 0, S = 0
    _diversity_both(B, orc, same, np.zeros(N, np.int32), N)
    u, t, d = B.as_ngram_diversity(torch.from_numpy(same).cuda(), torch.full((N,), 50, dtype=torch.int32, device="cuda"), N)
    assert t.cpu().tolist() == [[N * T, N * (T - 1), N * (T - 2), N * (T - 3)]]
    u, t, d = B.as_ngram_diversity(torch.empty((4, 0), dtype=torch.int32, device="cuda"),
                                   torch.zeros(4, dtype=torch.int32, device="cuda"), 2)
    assert t.cpu().numpy().sum() == 0 and d.cpu().tolist() == [0.0, 0.0]
    u, t, d = B.as_ngram_diversity(torch.empty((0, 5), dtype=torch.int32, device="cuda"),
                                   torch.empty(0, dtype=torch.int32, device="cuda"), 2)
    assert d.numel() == 0
    # a group that does not fit shared memory is refused, not mangled
    with pytest.raises(B.AsError) as e:
        B.as_ngram_diversity(torch.zeros((32, 1024), dtype=torch.int32, device="cuda"),
                             torch.zeros(32, dtype=torch.int32, device="cuda"), 32)
    assert e.value.code == B.ERR_UNSUPPORTED


def test_diversity_and_mean_of_oracle_decodes(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c1()
    table = w.table()
    ref = orc.decode_bigram(table, F32, w.starts(), w.N, w.shift(), w.T, w.eos, w.temp)
    seq, length = ref.seq.astype(np.int32), ref.len.astype(np.int32)
    _diversity_both(B, orc, seq, length, w.N)
    r = np.random.default_rng(3).normal(0, 1, w.V)
    lane, mean = B.as_reward_mean(torch.from_numpy(seq).cuda(), torch.from_numpy(length).cuda(), w.N,
                                  torch.from_numpy(r).cuda())
    wl, wm = orc.reward_mean(seq, length, w.N, r)
    np.testing.assert_allclose(lane.cpu().numpy(), wl, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(mean.cpu().numpy(), wm, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("S,N,T,V", [(1, 1, 1, 2), (9, 4, 7, 5), (64, 32, 128, 32128), (3, 1000, 33, 100), (5, 7, 600, 3)])
def test_reward_mean_random_tokens(B, orc, S, N, T, V):
    rng = np.random.default_rng(S + N + T)
    seq, length = _tokens(rng, S * N, T, V)
    r = rng.normal(0, 10, V) * (10.0 ** rng.integers(-3, 4, V))      # mixed magnitudes
    st = torch.empty(S, dtype=torch.int32, device="cuda")
    lane, mean = B.as_reward_mean(torch.from_numpy(seq).cuda(), torch.from_numpy(length).cuda(), N,
                                  torch.from_numpy(r).cuda(), group_status=st)
    torch.cuda.synchronize()
    wl, wm = orc.reward_mean(seq, length, N, r)
    scale = np.abs(r).max() * T
    np.testing.assert_allclose(lane.cpu().numpy(), wl, rtol=1e-12, atol=1e-13 * scale)
    np.testing.assert_allclose(mean.cpu().numpy(), wm, rtol=1e-12, atol=1e-13 * scale)
    assert (st.cpu().numpy() == 0).all()


def test_reward_mean_flags_tokens_outside_the_vocabulary(B):
    seq = torch.tensor([[0, 1, 2], [2, 9, 1], [1, 1, 1], [0, 0, -1]], dtype=torch.int32, device="cuda")
    ln = torch.tensor([3, 3, 3, 2], dtype=torch.int32, device="cuda")
    r = torch.tensor([1.0, 10.0, 100.0], dtype=torch.float64, device="cuda")
    st = torch.empty(2, dtype=torch.int32, device="cuda")
    lane, mean = B.as_reward_mean(seq, ln, 2, r, group_status=st)
    assert st.cpu().tolist() == [B.ERR_INVALID_ARG, 0]
    assert lane.cpu().tolist() == [111.0, 110.0, 30.0, 2.0] and mean.cpu().tolist() == [110.5, 16.0]


def test_estimator_has_zero_variance_on_a_lattice_matched_model(B):
    # Sec. 4.4, first proposition, through the GPU path alone: one step over 4 symbols with
    # probabilities 1/8, 3/8, 2/8, 2/8; with N = 8 codes every shift decodes the symbols 1, 3, 2, 2
    # times, so the sample mean equals the expectation whatever the shift
    p = np.array([1, 3, 2, 2]) / 8.0
    table = torch.from_numpy(np.tile(np.log(p).astype(np.float32), (4, 1))).cuda()
    r = np.array([0.25, -1.5, 4.0, 10.0])
    want = float((p * r).sum())
    starts = torch.zeros(3, dtype=torch.int32, device="cuda")
    for u in [0.013, 0.3, 0.5, 0.77, 0.999]:
        seq, ln = B.as_decode_bigram(table, starts, 8, u, 1, -1)
        lane, mean = B.as_reward_mean(seq, ln, 8, torch.from_numpy(r).cuda())
        assert mean.cpu().numpy() == pytest.approx(want, abs=1e-13)
        un, tot, d = B.as_ngram_diversity(seq, ln, 8)
        assert un.cpu().tolist() == [[4, 0, 0, 0]] * 3 and tot.cpu().tolist() == [[8, 0, 0, 0]] * 3


@pytest.mark.parametrize("N", [1, 2, 31, 256, 1000, 70001])
def test_lattice_variants_bit_exact(B, orc, N):
    for variant, b in [(0, 0.3), (1, 0.0), (1, 0.617), (1, 0.999999), (2, 0.0), (2, 0.4)]:
        got = B.as_lattice_codes_variant(N, b, variant).cpu().numpy()
        assert (got == orc.lattice_codes_variant(N, b, variant)).all()


def test_naive_codebook_bias_example_on_the_gpu(B):
    # the example after the proposition "Naive arithmetic sampling": N = 1 gives the code 0.5,
    # which decodes to the symbol of probability 0.6 every time
    table = torch.from_numpy(np.tile(np.log([0.6, 0.4, 1e-30, 1e-30]).astype(np.float32), (4, 1))).cuda()
    codes = B.as_lattice_codes_variant(1, 0.0, B.LATTICE_NAIVE)
    assert codes.cpu().tolist() == [0.5]
    seq, ln = B.as_decode_bigram_codes(table, torch.zeros(1, dtype=torch.int32, device="cuda"), codes, 1, -1)
    assert seq.cpu().tolist() == [[0]]
