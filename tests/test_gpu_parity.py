"""CUDA path vs CPU oracle, element by element, through the C-ABI binding (needs a B200)."""
import numpy as np
import pytest

from tests.parity import compare_step

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


def to_dev(arr, dtype):
    if dtype == BF16:
        return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).cuda()


def gpu_step(B, arr, dtype, codes, temp, top_k, top_p, V=None):
    d = {}
    tok, c2 = B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), temp, top_k, top_p, diag=d, V=V)
    torch.cuda.synchronize()
    return (tok.cpu().numpy(), c2.cpu().numpy(), d["p_tok"].cpu().numpy(), d["n_kept"].cpu().numpy(),
            d["lane_status"].cpu().numpy())


def check(B, orc, arr, dtype, codes, temp, top_k, top_p, V=None, what="", threads=8):
    ref = orc.step(arr, dtype, codes, temp, top_k, top_p, V=V, threads=threads)
    tok, c2, p, nk, st = gpu_step(B, arr, dtype, codes, temp, top_k, top_p, V=V)
    return compare_step(ref, tok, c2, p, nk, st, what=what)


MODS = [(1.0, 0, 1.0), (0.7, 5, 1.0), (1.3, 0, 0.9), (0.8, 7, 0.6), (0.5, 1, 1.0), (1.0, 0, 1e-6),
        (2.0, 1000000, 0.999)]


def _store(x, dtype):
    from paper_2210_15458_b200 import synth
    x = np.ascontiguousarray(x, dtype=np.float32)
    return synth.f32_to_bf16_bits(x) if dtype == BF16 else x


@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("V", [1, 2, 3, 5, 17, 33, 255, 1000, 4099, 9001])
def test_step_small_shapes_all_modifiers(B, orc, dtype, V):
    rng = np.random.default_rng(1000 + V)
    lanes = 37
    arr = _store(rng.normal(0, 3, (lanes, V)), dtype)
    codes = rng.random(lanes)
    codes[0] = 0.0
    codes[1] = 1.0
    codes[2] = 1.0 - 2.0 ** -53
    for temp, k, p in MODS:
        check(B, orc, arr, dtype, codes, temp, k, p, what="V=%d dt=%d mods=%s" % (V, dtype, (temp, k, p)))


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_heavy_ties(B, orc, dtype):
    # integer-valued logits: most elements tie at every threshold, so top-k and the nucleus
    # both cut inside groups of equal values (lowest indices win)
    rng = np.random.default_rng(77)
    for V in (64, 700, 5000):
        arr = _store(rng.integers(-3, 4, (29, V)), dtype)
        codes = rng.random(29)
        for temp, k, p in [(1.0, 10, 1.0), (0.9, 0, 0.5), (1.1, V // 2, 0.7), (1.0, 3, 0.99), (1.0, V - 1, 1.0)]:
            check(B, orc, arr, dtype, codes, temp, k, p, what="ties V=%d %s" % (V, (temp, k, p)))
    flat = _store(np.zeros((8, 3000)), dtype)                 # one value only
    check(B, orc, flat, dtype, rng.random(8), 1.0, 100, 0.5, what="flat row")


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_masked_and_nonfinite_lanes(B, orc, dtype):
    rng = np.random.default_rng(5)
    V = 777
    x = rng.normal(0, 2, (10, V)).astype(np.float32)
    x[0, ::2] = -np.inf
    x[1, :] = -np.inf
    x[1, 500] = 0.25                      # a single live token
    x[2, 3] = np.nan
    x[3, 700] = np.inf
    x[4, :] = -np.inf                     # empty row
    x[5, 10] = -np.nan
    arr = _store(x, dtype)
    codes = rng.random(10)
    codes[6] = 1.5
    codes[7] = np.nan
    codes[8] = -0.1
    for temp, k, p in [(1.0, 0, 1.0), (0.7, 4, 0.9)]:
        r = check(B, orc, arr, dtype, codes, temp, k, p, what="nonfinite")
    ref = orc.step(arr, dtype, codes)
    assert (ref.status[[2, 3, 4, 5, 6, 7, 8]] == orc.ERR_NUMERIC).all() and ref.status[[0, 1, 9]].tolist() == [0, 0, 0]
    tok, c2, *_ = gpu_step(B, arr, dtype, codes, 1.0, 0, 1.0)
    assert tok[1] == 500 and c2[6] == 1.5                      # code returned unchanged on failure


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_padded_and_unaligned_rows(B, orc, dtype):
    # ld > V, odd pitches (rows not 16-byte aligned) and a view that starts off-alignment
    rng = np.random.default_rng(9)
    for V, ld in [(1000, 1001), (1000, 1024), (33, 37), (4099, 4101)]:
        full = _store(rng.normal(0, 3, (21, ld)), dtype)
        codes = rng.random(21)
        check(B, orc, full, dtype, codes, 0.9, 6, 0.95, V=V, what="ld=%d" % ld)
    big = _store(rng.normal(0, 3, (12, 2051)), dtype)
    dev = to_dev(big, dtype)[:, 3:2003]                        # offset view, pitch 2051
    ref = orc.step(np.ascontiguousarray(big[:, 3:2003]), dtype, rng.random(12) * 0 + 0.37, 1.0, 9, 1.0)
    tok, c2 = B.as_step(dev, torch.full((12,), 0.37, dtype=torch.float64, device="cuda"), 1.0, 9, 1.0)
    compare_step(ref, tok.cpu().numpy(), c2.cpu().numpy(), what="offset view")


def test_step_in_place_and_deterministic(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c2()
    arr = w.logits(64)
    dev = to_dev(arr, BF16)
    codes = torch.from_numpy(orc.lattice_codes(64, 0.3)).cuda()
    t1, c1 = B.as_step(dev, codes, w.temp, w.top_k, w.top_p)
    t2, c2 = B.as_step(dev, codes, w.temp, w.top_k, w.top_p)
    assert torch.equal(t1, t2) and torch.equal(c1, c2)
    alias = codes.clone()
    t3, c3 = B.as_step(dev, alias, w.temp, w.top_k, w.top_p, codes_out=alias)
    assert torch.equal(t1, t3) and torch.equal(c1, alias)
    assert B.as_step(dev[:0], codes[:0], 1.0)[0].numel() == 0   # zero lanes is a no-op


def test_lattice_codes_bit_exact(B, orc):
    for N, u in [(1, 0.0), (7, 0.5), (256, 0.999999999), (1024, 1.0 - 2.0 ** -53), (100003, 0.123456789)]:
        got = B.as_lattice_codes(N, u).cpu().numpy()
        np.testing.assert_array_equal(got, orc.lattice_codes(N, u))
    with pytest.raises(B.AsError):
        B.as_lattice_codes(8, 1.0)


# --------------------------------------------------------------------------- the measured configurations
def test_c2_full(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c2()
    arr = w.logits()
    codes = orc.lattice_codes(w.N, w.shift())
    r = check(B, orc, arr, BF16, codes, w.temp, w.top_k, w.top_p, what="c2")
    assert r["compared"] > 0.95 * w.lanes
    iid = synth.iid_codes(w.lanes, 123)                      # ordinary ancestral sampling, same path
    check(B, orc, arr, BF16, iid, w.temp, w.top_k, w.top_p, what="c2 iid")


def _sampled_full_size(B, orc, w, sample, seed, extra=None):
    """The whole configuration through the CUDA path in the launch shape the benchmark times;
    `sample` lanes spread over the whole range (plus those `extra` picks from the GPU's own
    diagnostics) go through the oracle one by one; every lane gets range checks."""
    arr = w.logits()
    codes = orc.lattice_codes(w.N, w.shift())[: w.lanes]
    d = {}
    tok, c2 = B.as_step(to_dev(arr, w.dtype), torch.from_numpy(codes).cuda(), w.temp, w.top_k, w.top_p, diag=d)
    torch.cuda.synchronize()
    tok, c2 = tok.cpu().numpy(), c2.cpu().numpy()
    p, nk, st, path = (d[k].cpu().numpy() for k in ("p_tok", "n_kept", "lane_status", "path"))
    rng = np.random.default_rng(seed)
    # one lane from each of `sample` equal stretches: early and late rows of every persistent CTA
    edges = np.linspace(0, w.lanes, sample + 1).astype(np.int64)
    idx = set(int(rng.integers(edges[i], edges[i + 1])) for i in range(sample))
    if extra is not None:
        idx |= set(int(i) for i in extra(nk, path))
    idx = np.array(sorted(idx))
    ref = orc.step(np.ascontiguousarray(arr[idx]), w.dtype, codes[idx], w.temp, w.top_k, w.top_p, threads=8)
    r = compare_step(ref, tok[idx], c2[idx], p[idx], nk[idx], st[idx], what=w.name)
    assert (st == 0).all() and (tok >= 0).all() and (tok < w.V).all()
    assert (c2 >= 0).all() and (c2 < 1).all() and (nk >= 1).all()
    if w.top_k:
        assert (nk <= w.top_k).all()
    r["sampled"] = len(idx)
    return r


def test_c3_full_size_sampled(B, orc):
    from paper_2210_15458_b200 import synth

    def deep_lanes(nk, path):
        # the lanes with the largest kept sets are the ones whose nucleus reached below the first
        # threshold (the list was deepened) or that went to the general routine
        return list(np.argsort(-nk)[:24]) + list(np.nonzero(path == B.PATH_GENERAL)[0][:16])
    r = _sampled_full_size(B, orc, synth.c3(), 128, 1, extra=deep_lanes)
    assert r["sampled"] >= 128 and r["compared"] >= 0.9 * r["sampled"]


@pytest.mark.parametrize("lanes", [1024, 4096, 8192])
def test_c5_full_size_sampled(B, orc, lanes):
    from paper_2210_15458_b200 import synth
    r = _sampled_full_size(B, orc, synth.c5(lanes), 64, 2 + lanes)
    assert r["compared"] >= 56


@pytest.mark.parametrize("cluster", [4, 8])
def test_c5_rows_through_the_cluster_kernel(B, orc, cluster):
    # the row split over the CTAs of a thread-block cluster (slices in distributed shared memory)
    # at the full vocabulary of the large-vocabulary configuration
    from paper_2210_15458_b200 import synth
    w = synth.c5(96)
    arr = w.logits()
    codes = orc.lattice_codes(w.N, w.shift())
    try:
        B.as_tune(B.TUNE_STEP_PATH, 2)
        B.as_tune(B.TUNE_CLUSTER, cluster)
        r = check(B, orc, arr, BF16, codes, w.temp, w.top_k, w.top_p, what="c5 cluster=%d" % cluster)
        assert r["compared"] >= 88
    finally:
        B.as_tune(B.TUNE_CLUSTER, 0)
        B.as_tune(B.TUNE_STEP_PATH, 0)


# --------------------------------------------------------------------------- bigram decode loop
def _teacher_forced(B, orc, table, dtype, dev_table, prev, codes, T, eos, temp, top_k, top_p):
    """Oracle decodes freely and records each step's input state; the GPU then takes every
    recorded (previous token, code) as a one-step decode and must reproduce that step."""
    ref = orc.decode_bigram_codes(table, dtype, prev, codes, T, eos, temp, top_k, top_p, trace=True, threads=8)
    lanes = len(prev)
    ts = [(i, t) for i in range(lanes) for t in range(ref.len[i])]
    p_in = np.array([prev[i] if t == 0 else ref.seq[i, t - 1] for i, t in ts], np.int32)
    c_in = np.array([ref.trace_code_in[i, t] for i, t in ts])
    seq, ln = B.as_decode_bigram_codes(dev_table, torch.from_numpy(p_in).cuda(), torch.from_numpy(c_in).cuda(),
                                       1, eos, temp, top_k, top_p,
                                       codes_final=(cf := torch.empty(len(ts), dtype=torch.float64, device="cuda")))
    torch.cuda.synchronize()
    want_tok = np.array([ref.seq[i, t] for i, t in ts])
    want_c = np.array([ref.trace_code_out[i, t] for i, t in ts])
    d_tok = np.array([ref.trace_d_tok[i, t] for i, t in ts])
    safe = d_tok > 1e-5
    got = seq.cpu().numpy()[:, 0]
    assert (ln.cpu().numpy() == 1).all()
    assert (got[safe] == want_tok[safe]).all()
    np.testing.assert_allclose(cf.cpu().numpy()[safe], want_c[safe], rtol=1e-6, atol=1e-12)
    return ref, int(safe.sum()), len(ts)


def _comparable_prefix(ref, i):
    """Number of leading steps of lane i on which a free-running decode must still equal the
    oracle's: before the first step inside the boundary band, and while the rounding error of
    the code (~1e-16, multiplied by 1/p at every step) is still far below that band."""
    n = int(ref.len[i])
    amp = 1e-15
    for t in range(n):
        if not (ref.trace_d_tok[i, t] > 1e-5) or amp > 1e-8:
            return t
        amp /= ref.trace_p_tok[i, t]
    return n


def test_c1_decode(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c1()
    table = w.table()
    dev = to_dev(table, F32)
    starts = w.starts()
    u = w.shift()
    st = torch.empty(w.lanes, dtype=torch.int32, device="cuda")
    cf = torch.empty(w.lanes, dtype=torch.float64, device="cuda")
    seq, ln = B.as_decode_bigram(dev, torch.from_numpy(starts).cuda(), w.N, u, w.T, w.eos, w.temp,
                                 codes_final=cf, lane_status=st)
    torch.cuda.synchronize()
    prev = np.repeat(starts, w.N).astype(np.int32)
    codes = np.tile(orc.lattice_codes(w.N, u), w.S)
    ref, nsafe, nsteps = _teacher_forced(B, orc, table, F32, dev, prev, codes, w.T, w.eos, w.temp, 0, 1.0)
    assert nsafe > 0.98 * nsteps
    seq, ln = seq.cpu().numpy(), ln.cpu().numpy()
    assert (st.cpu().numpy() == 0).all()
    # free-running sequences agree up to the first step that sits in the boundary band
    compared = 0
    for i in range(w.lanes):
        upto = _comparable_prefix(ref, i)
        assert (seq[i, :upto] == ref.seq[i, :upto]).all()
        compared += upto
        assert (seq[i, ln[i]:] == -1).all() and (seq[i, :ln[i]] >= 0).all()
        if ln[i] < w.T:
            assert seq[i, ln[i] - 1] == w.eos
    assert compared >= 3 * w.lanes
    # split and resume: 16 steps == 8 + 8 from the returned state
    a_cf = torch.empty(w.lanes, dtype=torch.float64, device="cuda")
    a_seq, a_len = B.as_decode_bigram_codes(dev, torch.from_numpy(prev).cuda(), torch.from_numpy(codes).cuda(),
                                            8, w.eos, w.temp, codes_final=a_cf)
    alive = (a_len == 8) & (a_seq[:, 7] != w.eos)
    idx = torch.nonzero(alive)[:, 0]
    b_seq, b_len = B.as_decode_bigram_codes(dev, a_seq[idx, 7].contiguous(), a_cf[idx].contiguous(), 8, w.eos, w.temp)
    torch.cuda.synchronize()
    assert (b_seq.cpu().numpy() == seq[idx.cpu().numpy(), 8:]).all()


def test_decode_small_models_with_cuts_and_eos(B, orc):
    rng = np.random.default_rng(31)
    for dtype, V, eos, temp, k, p in [(F32, 50, 3, 1.0, 0, 1.0), (BF16, 300, 0, 0.8, 10, 1.0),
                                      (F32, 1000, 7, 1.2, 0, 0.8), (BF16, 2000, -1, 0.7, 20, 0.9)]:
        x = rng.normal(0, 2, (V, V)).astype(np.float32)
        if eos >= 0:
            x[:, eos] += 3.0                              # frequent EOS -> ragged lengths
        table = _store(x, dtype)
        dev = to_dev(table, dtype)
        prev = rng.integers(0, V, 96).astype(np.int32)
        codes = rng.random(96)
        ref, nsafe, nsteps = _teacher_forced(B, orc, table, dtype, dev, prev, codes, 12, eos, temp, k, p)
        assert nsafe > 0.9 * nsteps
        seq, ln = B.as_decode_bigram_codes(dev, torch.from_numpy(prev).cuda(), torch.from_numpy(codes).cuda(),
                                           12, eos, temp, k, p)
        seq, ln = seq.cpu().numpy(), ln.cpu().numpy()
        compared = 0
        for i in range(96):
            upto = _comparable_prefix(ref, i)
            assert (seq[i, :upto] == ref.seq[i, :upto]).all()
            if upto == ref.len[i]:
                assert ln[i] == ref.len[i] and (seq[i, upto:] == -1).all()
            compared += upto
        assert compared >= 96
    # T = 0 and an out-of-range start token
    seq, ln = B.as_decode_bigram_codes(dev, torch.tensor([1], dtype=torch.int32, device="cuda"),
                                       torch.tensor([0.5], dtype=torch.float64, device="cuda"), 0, -1)
    assert ln.cpu().item() == 0
    st = torch.empty(2, dtype=torch.int32, device="cuda")
    seq, ln = B.as_decode_bigram_codes(dev, torch.tensor([1, V + 5], dtype=torch.int32, device="cuda"),
                                       torch.tensor([0.5, 0.5], dtype=torch.float64, device="cuda"), 3, -1,
                                       lane_status=st)
    assert st.cpu().tolist() == [0, B.ERR_NUMERIC] and ln.cpu().tolist() == [3, 0]
    assert (seq[1].cpu().numpy() == -1).all()


def test_decode_lattice_properties_on_gpu_output(B, orc):
    # Sec. 4.3 on the GPU's own output: sorted codes give dictionary-ordered sequences, and a
    # first token of probability P is produced by floor(NP) or ceil(NP) lanes of a group.
    from paper_2210_15458_b200 import synth
    w = synth.c1()
    table = w.table()
    starts = w.starts()
    u = w.shift()
    seq, ln = B.as_decode_bigram(to_dev(table, F32), torch.from_numpy(starts).cuda(), w.N, u, w.T, w.eos, w.temp)
    seq = seq.cpu().numpy()
    for s in range(w.S):
        grp = [tuple(r) for r in seq[s * w.N:(s + 1) * w.N]]
        # codes of a group increase with j except for the wrap; after rotating, order is kept
        codes = orc.lattice_codes(w.N, u)
        order = np.argsort(codes, kind="stable")
        keyed = [tuple(np.where(np.array(grp[j]) < 0, 10 ** 6, np.array(grp[j]))) for j in order]
        # padded (-1) positions sort after every token except EOS itself, which ends the sequence
        firsts = [g[0] for g in keyed]
        assert firsts == sorted(firsts)
        row = table[starts[s]].astype(np.float64)
        pr = np.exp(row - row.max())
        pr /= pr.sum()
        cnt = np.bincount([g[0] for g in grp], minlength=w.V)
        assert (cnt >= np.floor(w.N * pr - 1e-9)).all() and (cnt <= np.ceil(w.N * pr + 1e-9)).all()


def test_c4_shape_reduced_table(B, orc):
    # c4's recipe (bf16 table, Zipf-like column bias, temperature 0.8, EOS id 1) on a 4096-token
    # vocabulary so that the whole loop runs in seconds; the full 32128 x 32128 table is
    # covered by test_c4_full_size_sampled.
    from paper_2210_15458_b200 import synth
    w = synth.c4(V=4096, S=16, T=48)
    table = w.table()
    dev = to_dev(table, BF16)
    prev = np.repeat(w.starts(), w.N).astype(np.int32)
    codes = np.tile(orc.lattice_codes(w.N, w.shift()), w.S)
    ref, nsafe, nsteps = _teacher_forced(B, orc, table, BF16, dev, prev, codes, w.T, w.eos, w.temp, 0, 1.0)
    assert nsafe > 0.97 * nsteps


def test_c4_full_size_sampled(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c4()
    table = w.table()
    dev = to_dev(table, BF16)
    starts = w.starts()
    u = w.shift()
    st = torch.empty(w.lanes, dtype=torch.int32, device="cuda")
    seq, ln = B.as_decode_bigram(dev, torch.from_numpy(starts).cuda(), w.N, u, w.T, w.eos, w.temp, lane_status=st)
    torch.cuda.synchronize()
    seq, ln = seq.cpu().numpy(), ln.cpu().numpy()
    assert (st.cpu().numpy() == 0).all() and (seq[np.arange(w.lanes), 0] >= 0).all()
    assert (seq < w.V).all()
    lanes = np.sort(np.random.default_rng(4).choice(w.lanes, 24, replace=False))
    prev = np.repeat(starts, w.N).astype(np.int32)[lanes]
    codes = np.tile(orc.lattice_codes(w.N, u), w.S)[lanes]
    ref, nsafe, nsteps = _teacher_forced(B, orc, table, BF16, dev, prev, codes, 24, w.eos, w.temp, 0, 1.0)
    assert nsafe > 0.97 * nsteps
    compared = 0
    for n, i in enumerate(lanes):
        upto = _comparable_prefix(ref, n)
        assert (seq[i, :upto] == ref.seq[n, :upto]).all()
        compared += upto
    assert compared >= 5 * len(lanes)
    # the same table with a cut: the loop then runs as one launch of the step kernel per step with
    # the rows gathered from the table (Sec. 5.1 "Top-k sampling"), teacher-forced against the oracle
    for k, p in [(10, 1.0), (0, 0.9), (40, 0.95)]:
        ref, nsafe, nsteps = _teacher_forced(B, orc, table, BF16, dev, prev[:12], codes[:12], 10, w.eos, w.temp, k, p)
        assert nsafe > 0.9 * nsteps and nsteps >= 100


# --------------------------------------------------------------------------- launch shapes
@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_every_cluster_size(B, orc, dtype, cluster):
    # the same lanes through 1, 2, 4 and 8 CTAs per lane (row slices in distributed shared
    # memory), with ragged tails, ties, and more lanes than resident clusters
    rng = np.random.default_rng(500 + cluster)
    try:
        B.as_tune(B.TUNE_STEP_PATH, 2)
        B.as_tune(B.TUNE_CLUSTER, cluster)
        for V, lanes in [(9001, 45), (40000, 300), (777, 20), (65536 + 24, 33)]:
            x = rng.normal(0, 3, (lanes, V)).astype(np.float32)
            x[:, : V // 3] = np.round(x[:, : V // 3])           # a third of the row is tie-prone
            arr = _store(x, dtype)
            codes = rng.random(lanes)
            for temp, k, p in [(0.7, 40, 1.0), (1.0, 0, 0.9), (0.8, 64, 0.95), (1.0, 0, 1.0), (1.0, 290, 0.5)]:
                check(B, orc, arr, dtype, codes, temp, k, p, what="cluster=%d V=%d %s" % (cluster, V, (temp, k, p)))
    finally:
        B.as_tune(B.TUNE_CLUSTER, 0)
        B.as_tune(B.TUNE_STEP_PATH, 0)


@pytest.mark.parametrize("stages", [2, 3, 5])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_streamed_rows(B, orc, dtype, stages):
    # rows longer than the shared-memory ring: slices stream through 2, 3 or 5 stages, the
    # threshold is refreshed at slices 0, 1, 2, 4, ..., ragged last slice and ragged last vector
    rng = np.random.default_rng(700 + stages)
    try:
        B.as_tune(B.TUNE_STAGES, stages)
        for V, lanes in [(70001, 40), (131072, 12), (200003, 9)]:
            x = rng.normal(0, 3, (lanes, V)).astype(np.float32)
            x[:, ::3] = np.round(x[:, ::3])
            x[: lanes // 2] += np.linspace(0, 6, V, dtype=np.float32)[None, :]   # the best tokens come last
            arr = _store(x, dtype)
            codes = rng.random(lanes)
            for temp, k, p in [(0.7, 40, 1.0), (1.0, 0, 0.9), (0.8, 64, 0.95), (1.0, 128, 0.5), (1.0, 1, 1.0)]:
                check(B, orc, arr, dtype, codes, temp, k, p, what="stages=%d V=%d %s" % (stages, V, (temp, k, p)))
    finally:
        B.as_tune(B.TUNE_STAGES, 0)


def test_step_general_path_only(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c2()
    arr = w.logits(96)
    codes = orc.lattice_codes(96, 0.77)
    try:
        B.as_tune(B.TUNE_STEP_PATH, 1)
        check(B, orc, arr, BF16, codes, w.temp, w.top_k, 0.9, what="general path")
    finally:
        B.as_tune(B.TUNE_STEP_PATH, 0)


def test_step_flat_and_adversarial_rows_fall_back(B, orc):
    # rows the compaction cannot serve: everything ties with the maximum, a nucleus that needs
    # most of the vocabulary, top-k larger than the candidate capacity
    rng = np.random.default_rng(600)
    V = 20000
    flat = _store(np.zeros((6, V)), BF16)
    check(B, orc, flat, BF16, rng.random(6), 1.0, 40, 1.0, what="flat top-k")
    check(B, orc, flat, BF16, rng.random(6), 1.0, 0, 0.9, what="flat nucleus")
    wide = _store(rng.normal(0, 0.05, (6, V)), F32)
    check(B, orc, wide, F32, rng.random(6), 1.0, 0, 0.97, what="wide nucleus")
    check(B, orc, wide, F32, rng.random(6), 1.0, 5000, 1.0, what="large top-k")
    check(B, orc, wide, F32, rng.random(6), 1.0, 5000, 0.3, what="large top-k + nucleus")


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_wide_nucleus_through_value_bins(B, orc, dtype):
    # nuclei of hundreds to tens of thousands of tokens (flat rows), with ties at the threshold,
    # masked tokens and unaligned rows: the general routine settles them through bins of the logit
    # value; the same lanes through its radix select must give the very same tokens and kept counts
    rng = np.random.default_rng(4242)
    cases = [(128256, 3.0, 0.8, 0.9), (50001, 1.0, 1.0, 0.5), (50001, 0.05, 1.0, 0.97),
             (32000, 3.0, 2.0, 0.99), (9001, 2.0, 1.0, 0.3), (4099, 1.5, 1.0, 0.8)]
    for V, sigma, temp, p in cases:
        lanes = 10
        x = rng.normal(0, sigma, (lanes, V)).astype(np.float32)
        x[1, ::3] = -np.inf                                       # masked tokens
        x[2] = np.round(x[2] * 2) / 2                             # few distinct values: ties everywhere
        arr = _store(x, dtype)
        codes = rng.random(lanes)
        codes[3] = 0.0
        codes[4] = 1.0 - 2.0 ** -53
        ref = orc.step(arr, dtype, codes, temp, 0, p, threads=8)
        assert V < 32000 or np.median(ref.n_kept) > 300
        got = {}
        for name, key, val in [("default", None, 0), ("general", B.TUNE_STEP_PATH, 1)]:
            for radix in (0, 1):
                try:
                    if key is not None:
                        B.as_tune(key, val)
                    B.as_tune(B.TUNE_RADIX_NUCLEUS, radix)
                    tok, c2, pt, nk, st = gpu_step(B, arr, dtype, codes, temp, 0, p)
                finally:
                    B.as_tune(B.TUNE_RADIX_NUCLEUS, 0)
                    if key is not None:
                        B.as_tune(key, 0)
                what = "wide nucleus V=%d %s radix=%d" % (V, name, radix)
                compare_step(ref, tok, c2, pt, nk, st, what=what)
                # with tens of thousands of kept tokens every code lies within the usual band of a CDF
                # boundary; both sides compute in fp64, so a band of 1e-9 still leaves rounding room
                near = (ref.d_tok > 1e-9) & (ref.d_topp > 1e-9) & (ref.status == 0)
                assert near.sum() >= lanes - 2, what
                assert (tok[near] == ref.tokens[near]).all(), what
                assert (nk[near] == ref.n_kept[near]).all(), what
                np.testing.assert_allclose(pt[near], ref.p_tok[near], rtol=1e-9, err_msg=what)
                np.testing.assert_allclose(c2[near], ref.codes[near], rtol=0, atol=1e-5, err_msg=what)
                got[(name, radix)] = (tok, nk, c2)
        for name in ("default", "general"):
            assert (got[(name, 0)][0] == got[(name, 1)][0]).all() and (got[(name, 0)][1] == got[(name, 1)][1]).all()
            np.testing.assert_allclose(got[(name, 0)][2], got[(name, 1)][2], rtol=0, atol=1e-6)
    # rows off the 16-byte grid (element-wise loads in the general routine)
    full = _store(rng.normal(0, 1.0, (9, 6007)), dtype)
    try:
        B.as_tune(B.TUNE_STEP_PATH, 1)
        check(B, orc, full, dtype, rng.random(9), 1.0, 0, 0.9, V=6001, what="wide nucleus, odd pitch")
    finally:
        B.as_tune(B.TUNE_STEP_PATH, 0)


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_nucleus_deeper_than_the_list(B, orc, dtype):
    # nucleus-only lanes whose nucleus holds a few hundred tokens: more than the exact depth of the
    # candidate list, so the threshold has to be lowered once from the mass histogram; plus lanes
    # whose nucleus is far too large for any list (general routine)
    rng = np.random.default_rng(800)
    for V in (50000, 140000):
        lanes = 24
        x = rng.normal(-12.0, 1.0, (lanes, V)).astype(np.float32)
        for i in range(lanes):
            n_hi = 120 + 20 * i                                   # 120 .. 580 comparable heavy tokens
            idx = rng.choice(V, n_hi, replace=False)
            x[i, idx] = rng.normal(2.0, 0.6, n_hi).astype(np.float32)
        arr = _store(x, dtype)
        codes = rng.random(lanes)
        d = {}
        ref = orc.step(arr, dtype, codes, 1.0, 0, 0.9, threads=8)
        tok, c2 = B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), 1.0, 0, 0.9, diag=d)
        torch.cuda.synchronize()
        r = compare_step(ref, tok.cpu().numpy(), c2.cpu().numpy(), d["p_tok"].cpu().numpy(),
                         d["n_kept"].cpu().numpy(), d["lane_status"].cpu().numpy(), what="deep nucleus V=%d" % V)
        assert r["compared"] >= lanes - 4
        path = d["path"].cpu().numpy()
        assert ref.n_kept.max() > 300
        assert (path[ref.n_kept < 400] == B.PATH_COMPACT).sum() >= 8    # served without the general routine


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_hit_list_overflow_takes_one_more_pass(B, orc, dtype):
    # rows whose level rises from one 16 KB slice to the next: between two refreshes of the
    # threshold a large share of the vectors beats the stale value, so the hit list overflows;
    # the final threshold is exact all the same and the candidates are taken in a second pass
    # over the row, without the general routine
    rng = np.random.default_rng(900)
    per_slice = 4096 if dtype == F32 else 8192
    V = 36 * per_slice + 1232                                  # row pitch stays a multiple of 16 bytes
    lanes = 12
    x = rng.normal(0, 3, (lanes, V)).astype(np.float32)
    x += (np.arange(V) // per_slice).astype(np.float32) * 0.45
    arr = _store(x, dtype)
    codes = rng.random(lanes)
    for temp, k, p in [(1.0, 40, 1.0), (0.8, 0, 0.9), (1.0, 64, 0.95)]:
        d = {}
        ref = orc.step(arr, dtype, codes, temp, k, p, threads=8)
        tok, c2 = B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), temp, k, p, diag=d)
        torch.cuda.synchronize()
        compare_step(ref, tok.cpu().numpy(), c2.cpu().numpy(), d["p_tok"].cpu().numpy(),
                     d["n_kept"].cpu().numpy(), d["lane_status"].cpu().numpy(),
                     what="overflow %s" % ((temp, k, p),))
        assert (d["path"].cpu().numpy() == B.PATH_COMPACT).sum() >= lanes // 2 + 1


@pytest.mark.parametrize("dtype,V", [(BF16, 32000), (F32, 5000), (BF16, 140000), (F32, 33)])
def test_step_lattice_equals_lattice_codes_then_step(B, orc, dtype, V):
    # codes formed in the kernel are the very values as_lattice_codes writes: the fused first step
    # must reproduce the two-call result bit for bit, on every kernel path, also for a slice j0..
    rng = np.random.default_rng(V)
    N, lanes, j0, u = 97, 40, 31, 0.8125
    arr = _store(rng.normal(0, 3, (lanes, V)), dtype)
    dev = to_dev(arr, dtype)
    codes = B.as_lattice_codes(N, u)
    for temp, k, p in [(0.7, 40, 1.0), (1.0, 0, 0.9), (1.0, 0, 1.0)]:
        tok_a, c_a = B.as_step(dev, codes[j0:j0 + lanes].contiguous(), temp, k, p)
        tok_b, c_b = B.as_step_lattice(dev, N, u, j0, temp, k, p)
        torch.cuda.synchronize()
        assert (tok_a == tok_b).all() and (c_a == c_b).all()
    check(B, orc, arr, dtype, orc.lattice_codes(N, u)[j0:j0 + lanes], 0.7, 40, 1.0, what="lattice slice")
    try:
        B.as_tune(B.TUNE_STEP_PATH, 2)
        tok_a, c_a = B.as_step(dev, codes[j0:j0 + lanes].contiguous(), 0.7, 40, 1.0)
        tok_b, c_b = B.as_step_lattice(dev, N, u, j0, 0.7, 40, 1.0)
        assert (tok_a == tok_b).all() and (c_a == c_b).all()
    finally:
        B.as_tune(B.TUNE_STEP_PATH, 0)


@pytest.mark.parametrize("dtype,V,ld", [(BF16, 32001, 32001), (F32, 5003, 5003), (BF16, 32000, 32000), (BF16, 4097, 4100)])
def test_step_host_buffers_any_pitch(B, orc, dtype, V, ld):
    # host buffers whose pitch is not a multiple of 16 bytes are staged at an aligned pitch
    rng = np.random.default_rng(V + ld)
    lanes = 24
    full = _store(rng.normal(0, 3, (lanes, ld)), dtype)
    arr = np.ascontiguousarray(full[:, :V])
    codes = rng.random(lanes)
    ref = orc.step(arr, dtype, codes, 0.8, 30, 0.95, threads=8)
    h_logits = torch.from_numpy(full.view(np.int16)).view(torch.bfloat16) if dtype == BF16 else torch.from_numpy(full)
    h_codes = torch.from_numpy(codes)
    tok = torch.empty(lanes, dtype=torch.int32)
    c2 = torch.empty(lanes, dtype=torch.float64)
    st = torch.empty(lanes, dtype=torch.int32)
    work = torch.empty(B.as_step_host_work_bytes(dtype, lanes, ld) + 256, dtype=torch.uint8, device="cuda")
    B.as_step_host(h_logits, h_codes, 0.8, 30, 0.95, tok, c2, st, work, V=V)
    r = compare_step(ref, tok.numpy(), c2.numpy(), status=st.numpy(), what="host buffers V=%d ld=%d" % (V, ld))
    assert r["compared"] >= lanes - 3


@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("V,pad", [(32001, 0), (4099, 3), (200003, 2), (140001, 0), (63, 0)])
def test_step_rows_off_the_16_byte_grid_take_the_fast_path(B, orc, dtype, V, pad):
    # a pitch that is only element-aligned: most rows start inside a 16-byte granule.  They are
    # copied from the granule's start and the elements in front are masked -- which this test
    # makes as tempting as possible: the padding between rows holds huge values, and the row's
    # own first and last elements are its largest.
    rng = np.random.default_rng(V + pad)
    lanes = 19
    ld = V + pad
    x = rng.normal(0, 3, (lanes, ld)).astype(np.float32)
    x[:, V:] = 80.0
    x[:, 0] += 9.0
    x[:, V - 1] += 9.0
    full = _store(x, dtype)
    off = 3                                               # the base pointer itself is off the grid too
    flat = np.concatenate([_store(np.full(off, 90.0, np.float32), dtype), full.ravel()])
    dev_flat = to_dev(flat, dtype)
    dev = dev_flat[off:].view(lanes, ld)
    arr = np.ascontiguousarray(full[:, :V])
    codes = rng.random(lanes)
    codes[0], codes[1] = 0.0, 1.0
    for temp, k, p in [(0.7, 40, 1.0), (0.5, 0, 0.9), (0.9, 64, 0.95), (1.0, 1, 1.0)]:
        d = {}
        ref = orc.step(arr, dtype, codes, temp, k, p, threads=8)
        tok, c2 = B.as_step(dev, torch.from_numpy(codes).cuda(), temp, k, p, diag=d, V=V)
        torch.cuda.synchronize()
        compare_step(ref, tok.cpu().numpy(), c2.cpu().numpy(), d["p_tok"].cpu().numpy(), d["n_kept"].cpu().numpy(),
                     d["lane_status"].cpu().numpy(), what="off-grid rows V=%d %s" % (V, (temp, k, p)))
        if V >= 4099:
            assert (d["path"].cpu().numpy() == B.PATH_COMPACT).sum() >= lanes - 3
    # no cut at all: the general routine, still correct
    check(B, orc, arr[:4], dtype, codes[:4], 1.0, 0, 1.0, what="off-grid rows, no cut")


@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("V", [2, 5, 24, 200, 4096 + 40])
def test_step_rows_with_fewer_tokens_than_the_cut_asks_for(B, orc, dtype, V):
    # fewer finite tokens than top_k (or than the list aims at): the threshold falls to -inf.  Only
    # vectors that exist may then count as hits: the ring holds one stage for such a row, and the
    # space behind a short row is whatever the previous launch left there.  The list must decide
    # these lanes itself (no detour through the general routine), masked tokens staying out.
    rng = np.random.default_rng(300 + V)
    lanes = 21
    x = rng.normal(0, 3, (lanes, V)).astype(np.float32)
    if V > 8:
        x[:, rng.choice(V, V // 3, replace=False)] = -np.inf
    arr = _store(x, dtype)
    codes = rng.random(lanes)
    codes[0], codes[1] = 0.0, 1.0
    dev = to_dev(arr, dtype)                               # aligned rows when V * size is a multiple of 16
    for temp, k, p in [(1.0, 1, 1.0), (0.8, V - 1 if V > 2 else 1, 1.0), (0.7, min(V - 1, 250), 0.9), (1.2, 0, 0.6)]:
        if k > 256:
            continue
        d = {}
        ref = orc.step(arr, dtype, codes, temp, k, p, threads=8)
        tok, c2 = B.as_step(dev, torch.from_numpy(codes).cuda(), temp, k, p, diag=d)
        torch.cuda.synchronize()
        compare_step(ref, tok.cpu().numpy(), c2.cpu().numpy(), d["p_tok"].cpu().numpy(), d["n_kept"].cpu().numpy(),
                     d["lane_status"].cpu().numpy(), what="short rows V=%d %s" % (V, (temp, k, p)))
        if k > 0:
            assert (d["path"].cpu().numpy() == B.PATH_COMPACT).all()


def test_step_overlapped_launches_give_the_same_results(B):
    # launches of one row per CTA may start while the launch before them drains (programmatic
    # dependent launch): a chain of steps, each reading the codes the one before wrote, must give
    # bit for bit what the same chain gives as ordinary launches
    from paper_2210_15458_b200 import synth
    w = synth.StepWorkload("chain", lanes=200, V=32000, dtype=synth.BF16, sigma=3.0, temp=0.7, top_k=40,
                           top_p=1.0, seed_logits=71, seed_perm=72, seed_shift=73)
    logits = to_dev(w.logits(), BF16)
    results = []
    for serial in (1, 0):
        B.as_tune(B.TUNE_SERIAL_LAUNCH, serial)
        try:
            codes = B.as_lattice_codes(w.N, w.shift())
            toks = torch.empty((12, w.lanes), dtype=torch.int32, device="cuda")
            for t in range(12):                      # back to back, no host synchronisation between
                B.as_step(logits, codes, w.temp, w.top_k, w.top_p, tokens=toks[t], codes_out=codes)
            torch.cuda.synchronize()
            results.append((toks.cpu().numpy(), codes.cpu().numpy()))
        finally:
            B.as_tune(B.TUNE_SERIAL_LAUNCH, 0)
    assert np.array_equal(results[0][0], results[1][0])
    assert np.array_equal(results[0][1], results[1][1])


def test_decode_with_cuts_per_step_kernels_equal_the_single_kernel(B, orc):
    # with a cut and a codes_final buffer the loop runs as one launch of the step kernel per step
    # (rows gathered from the table); without the buffer, as one general kernel.  Both follow the
    # same arithmetic up to rounding: sequences agree wherever the oracle's margins are safe.
    rng = np.random.default_rng(77)
    for dtype, V, ld, eos, temp, k, p in [(BF16, 3000, 3000, 5, 0.8, 12, 1.0), (F32, 2001, 2003, -1, 1.1, 0, 0.85),
                                          (BF16, 70001, 70001, 0, 0.7, 40, 0.95)]:
        x = rng.normal(0, 2.5, (V, ld)).astype(np.float32)
        if eos >= 0:
            x[:, eos] += 4.0
        table = _store(x, dtype)
        dev = to_dev(table, dtype)
        lanes, T = 40, 10
        prev = rng.integers(0, V, lanes).astype(np.int32)
        prev[3] = V + 7                                             # out of range: status, no tokens
        codes = rng.random(lanes)
        outs = []
        for per_step in (True, False):
            st = torch.empty(lanes, dtype=torch.int32, device="cuda")
            cf = torch.empty(lanes, dtype=torch.float64, device="cuda") if per_step else None
            seq, ln = B.as_decode_bigram_codes(dev, torch.from_numpy(prev).cuda(), torch.from_numpy(codes).cuda(), T,
                                               eos, temp, k, p, V=V, codes_final=cf, lane_status=st, per_step=per_step)
            torch.cuda.synchronize()
            outs.append((seq.cpu().numpy(), ln.cpu().numpy(), st.cpu().numpy()))
        (s1, l1, t1), (s2, l2, t2) = outs
        assert t1[3] == B.ERR_NUMERIC and t2[3] == B.ERR_NUMERIC and l1[3] == 0 and (s1[3] == -1).all()
        # the first tokens can only differ inside the boundary band; count whole-prefix agreement
        agree = [(s1[i, :4] == s2[i, :4]).all() for i in range(lanes)]
        assert np.mean(agree) > 0.9
        for i in range(lanes):
            assert (s1[i, l1[i]:] == -1).all() and (s1[i, :l1[i]] >= 0).all()
            if 0 < l1[i] < T:
                assert s1[i, l1[i] - 1] == eos


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_signed_zeros_tie_and_fall_to_the_lower_index(B, orc, dtype):
    # -0.0 and +0.0 are the same logit: where a top-k or nucleus boundary falls between them the
    # lower index wins, whatever the signs
    rng = np.random.default_rng(12)
    V, lanes = 4099, 16
    x = rng.normal(-4, 1, (lanes, V)).astype(np.float32)
    for i in range(lanes):
        z = rng.choice(V, 6, replace=False)
        x[i, z] = np.where(rng.random(6) < 0.5, -0.0, 0.0).astype(np.float32)   # the six largest, signs mixed
    x[0, :2] = [-0.0, 0.0]
    arr = _store(x, dtype)
    codes = rng.random(lanes)
    for temp, k, p in [(1.0, 1, 1.0), (1.0, 3, 1.0), (0.8, 0, 0.4), (1.0, 5, 0.5)]:
        check(B, orc, arr, dtype, codes, temp, k, p, what="signed zeros %s" % ((temp, k, p),))
    tok, _ = B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), 1.0, 1, 1.0)
    ref = orc.step(arr, dtype, codes, 1.0, 1, 1.0)
    assert np.array_equal(tok.cpu().numpy(), ref.tokens)           # top_k = 1: no band, exact


@pytest.mark.parametrize("path,V", [(0, 32000), (0, 140000), (2, 40000)])
def test_a_wait_that_runs_out_reports_timeout_and_the_next_call_is_fine(B, orc, path, V):
    # every wait for a copy is bounded.  With the copy-issuing thread told to issue nothing (so no
    # copy is in flight) and a limit of a million cycles, the wait runs out: the lane must come back
    # with AS_ERR_TIMEOUT, token -1 and its code unchanged, the kernel returns normally, and the
    # next ordinary call gives the oracle's result.
    rng = np.random.default_rng(V)
    arr = _store(rng.normal(0, 3, (3, V)), BF16)
    dev = to_dev(arr, BF16)
    codes = np.array([0.25, 0.5, 0.75])
    try:
        B.as_tune(B.TUNE_STEP_PATH, path)
        B.as_tune(B.TUNE_WAIT_KCYCLES, 1000)
        B.as_tune(B.TUNE_DEBUG_NO_COPY, 1)
        d = {}
        tok, c2 = B.as_step(dev, torch.from_numpy(codes).cuda(), 0.8, 20, 1.0, diag=d)
        torch.cuda.synchronize()
        assert (d["lane_status"].cpu().numpy() == B.ERR_TIMEOUT).all()
        assert (tok.cpu().numpy() == -1).all() and np.array_equal(c2.cpu().numpy(), codes)
    finally:
        B.as_tune(B.TUNE_DEBUG_NO_COPY, 0)
        B.as_tune(B.TUNE_WAIT_KCYCLES, 0)
    try:
        check(B, orc, arr, BF16, codes, 0.8, 20, 1.0, what="after a time-out")
    finally:
        B.as_tune(B.TUNE_STEP_PATH, 0)


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_without_a_cut_every_evaluation_mode(B, orc, dtype):
    # temperature only (Algorithm 1 as stated): rows in shared memory, masses from the bf16 table
    # or from the fp64 exponential.  Covered: ragged row ends, rows of one piece and of several,
    # masked tokens, zeros of both signs and subnormals (outside the table: evaluated directly),
    # magnitudes >= 64 (the row is redone relative to its maximum), temperatures below the
    # table's range, NaN / +inf / all-masked rows, codes 0 and 1.
    rng = np.random.default_rng(4242)
    for V, ld in [(8, 8), (64, 64), (4099, 4104), (9000, 9000), (32128, 32128), (49152, 49152), (40003, 40008)]:
        lanes = 23
        x = rng.normal(0, 2.5, (lanes, ld)).astype(np.float32)
        x[:, V:] = 70.0                                        # padding between rows must not count
        x[1, : V // 2] = -np.inf
        x[2, rng.choice(V, max(1, V // 7), replace=False)] = 0.0
        x[2, rng.choice(V, max(1, V // 9), replace=False)] = -0.0
        x[3, rng.choice(V, max(1, V // 5), replace=False)] = 1e-39    # subnormal in fp32, zero in bf16
        x[4, rng.integers(0, V)] = 77.0                        # outside the table: robust pass
        x[5, :] -= 300.0                                       # everything far below zero
        x[6, rng.integers(0, V)] = np.nan
        x[7, rng.integers(0, V)] = np.inf
        x[8, :] = -np.inf
        x[9, :] = -np.inf
        x[9, V - 1] = -5.0                                     # a single live token, the last one
        x[10, :] = 3.0                                         # flat row
        arr = _store(x, dtype)
        codes = rng.random(lanes)
        codes[0], codes[11], codes[12] = 0.0, 1.0, 1.0 - 2.0 ** -53
        codes[13] = 1.5
        for temp in (0.8, 1.0, 0.05, 3.0):
            r = check(B, orc, arr, dtype, codes, temp, 0, 1.0, V=V, what="no cut V=%d dt=%d temp=%g" % (V, dtype, temp))
            # (at temperature 3 a long row is nearly flat: most tokens are narrower than the boundary band)
            assert r["compared"] >= (8 if temp < 2.0 or V < 4000 else 3)


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_typical_cut(B, orc, dtype):
    # the locally typical set in place of the nucleus (Sec. 2 names typical decoding among the logit
    # modifiers): small and ragged shapes, tie-heavy rows (equal logits are equally typical: the lower
    # indices stay), masked tokens, a preceding top-k, and a Zipf-like 32000-token row
    from paper_2210_15458_b200 import synth
    rng = np.random.default_rng(2024)
    cases = []
    for V in (2, 5, 33, 1000, 4099):
        x = rng.normal(0, 2.5, (19, V)).astype(np.float32)
        if V > 8:
            x[3, rng.choice(V, V // 4, replace=False)] = -np.inf
            x[4:8] = np.round(x[4:8])
        cases.append(x)
    cases.append(np.zeros((6, 3000), np.float32))                          # flat: ties everywhere
    for x in cases:
        arr = _store(x, dtype)
        lanes = arr.shape[0]
        codes = rng.random(lanes)
        codes[0], codes[1] = 0.0, 1.0
        for temp, k, tp in [(1.0, 0, 0.9), (0.7, 0, 0.5), (1.3, 6, 0.8), (1.0, 0, 0.2), (0.9, 40, 0.95)]:
            ref = orc.step(arr, dtype, codes, temp, k, typical_p=tp, threads=8)
            d = {}
            tok, c2 = B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), temp, k, diag=d, typical_p=tp)
            torch.cuda.synchronize()
            compare_step(ref, tok.cpu().numpy(), c2.cpu().numpy(), d["p_tok"].cpu().numpy(), d["n_kept"].cpu().numpy(),
                         d["lane_status"].cpu().numpy(), what="typical V=%d %s" % (arr.shape[1], (temp, k, tp)))
    w = synth.c2()
    arr = w.logits(48) if dtype == BF16 else synth.bf16_bits_to_f32(w.logits(48))
    codes = orc.lattice_codes(48, 0.41)
    for temp, k, tp in [(0.7, 0, 0.9), (1.0, 0, 0.5), (0.7, 200, 0.95)]:
        ref = orc.step(arr, dtype, codes, temp, k, typical_p=tp, threads=8)
        d = {}
        tok, c2 = B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), temp, k, diag=d, typical_p=tp)
        torch.cuda.synchronize()
        r = compare_step(ref, tok.cpu().numpy(), c2.cpu().numpy(), d["p_tok"].cpu().numpy(), d["n_kept"].cpu().numpy(),
                         d["lane_status"].cpu().numpy(), what="typical c2 rows %s" % ((temp, k, tp),))
        assert r["compared"] >= 36
    with pytest.raises(ValueError):
        B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), 1.0, 0, 0.9, typical_p=0.5)


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_codes_at_the_top_end_through_the_general_routine(B, orc, dtype):
    # a code of 1 (or the largest double below it) selects the last kept token.  With few kept tokens
    # spread over a long row, most chunks of the row hold no mass; which chunk is the last one with
    # mass must not be read off rounded prefix sums
    rng = np.random.default_rng(4711)
    for V in (9001, 40000, 200003):
        lanes = 24
        arr = _store(rng.normal(0, 3, (lanes, V)), dtype)
        for c in (1.0, 1.0 - 2.0 ** -53, 0.0):
            codes = np.full(lanes, c)
            for temp, k, p in [(1.0, 300, 0.5), (1.0, 4, 1.0), (0.9, 0, 0.3), (1.0, 1000, 0.2)]:
                try:
                    B.as_tune(B.TUNE_STEP_PATH, 1)
                    ref = orc.step(arr, dtype, codes, temp, k, p, threads=8)
                    d = {}
                    tok, c2 = B.as_step(to_dev(arr, dtype), torch.from_numpy(codes).cuda(), temp, k, p, diag=d)
                    torch.cuda.synchronize()
                finally:
                    B.as_tune(B.TUNE_STEP_PATH, 0)
                st = d["lane_status"].cpu().numpy()
                assert (st == 0).all(), "V=%d code %r %s: status %s" % (V, c, (temp, k, p), st)
                # at the very ends the token is the first / last kept one whatever the rounding
                sure = ref.d_topp > 1e-6
                assert np.array_equal(tok.cpu().numpy()[sure], ref.tokens[sure])
                assert np.array_equal(d["n_kept"].cpu().numpy()[sure], ref.n_kept[sure])
