"""Extended-precision codes on the GPU against the oracle's exact decoder (needs a B200)."""
from fractions import Fraction

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


def to_dev(arr, dtype):
    if dtype == BF16:
        return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).cuda()


def _store(x, dtype):
    from paper_2210_15458_b200 import synth
    x = np.ascontiguousarray(x, dtype=np.float32)
    return synth.f32_to_bf16_bits(x) if dtype == BF16 else x


def _state_to_dev(st):
    return torch.from_numpy(st.view(np.int64).copy()).cuda()


def _state_from_dev(t):
    return t.cpu().numpy().view(np.uint64)


def test_lattice_state_bit_exact(B, orc):
    for N, u, j0, count, S in [(1, 0.0, 0, 1, 1), (7, 0.5, 0, 7, 3), (1000, 1.0 - 2.0 ** -53, 17, 400, 2),
                               (2 ** 31 - 1, 0.123456789, 2 ** 31 - 50, 49, 1), (100003, 1e-300, 0, 100003, 1)]:
        got = _state_from_dev(B.as_xp_lattice_state(N, u, j0, count, S))
        np.testing.assert_array_equal(got, orc.xp_lattice_state(N, u, S, j0, count))
    with pytest.raises(B.AsError):
        B.as_xp_lattice_state(8, 1.0)
    with pytest.raises(B.AsError):
        B.as_xp_lattice_state(8, 0.5, 5, 4)


def test_binary_digits_of_the_codes(B):
    # two equally likely tokens: the decoded tokens are the binary digits of (j + u)/N, for ever
    table = torch.zeros((2, 8), dtype=torch.float32, device="cuda")
    for N, u in [(3, 0.7), (1000, 0.123456789), (2 ** 31 - 1, 0.5)]:
        js = [0, N // 3, N - 1]
        st = torch.cat([B.as_xp_lattice_state(N, u, j, 1) for j in js])
        seq, ln = B.as_decode_bigram_xp(table, torch.zeros(3, dtype=torch.int32, device="cuda"), st, N, 200, -1, V=2)
        for row, j in zip(seq.cpu().numpy(), js):
            c = Fraction(j * (1 << 53) + int(np.floor(u * 2.0 ** 53)), N * (1 << 53))
            assert row.tolist() == [int(c * (1 << (t + 1))) & 1 for t in range(200)]


def _teacher_forced(B, orc, table, dtype, dev, prev0, st0, N, T, eos, temp, k, p):
    """The oracle decodes step by step and records each step's input; the GPU takes every recorded
    (previous token, state) as a one-step decode and must reproduce the step."""
    lanes = len(prev0)
    prevs, states, toks, news, dts = [], [], [], [], []
    prev, st = prev0.copy(), st0.copy()
    alive = np.ones(lanes, bool)
    for t in range(T):
        o = orc.xp_decode_bigram(table, dtype, prev, st, N, 1, eos, temp, k, p, trace=True, threads=8)
        idx = np.nonzero(alive & (o.status == 0) & (o.len == 1))[0]
        prevs.append(prev[idx].copy()); states.append(st[idx].copy()); toks.append(o.seq[idx, 0].copy())
        news.append(o.state[idx].copy()); dts.append(o.trace_d_tok[idx, 0].copy())
        alive &= (o.status == 0) & (o.len == 1) & (o.seq[:, 0] != eos)
        prev = np.where(alive, o.seq[:, 0], prev).astype(np.int32)
        st = o.state
    prevs, states, toks, news, dts = (np.concatenate(x) for x in (prevs, states, toks, news, dts))
    d_state = _state_to_dev(states)
    seq, ln = B.as_decode_bigram_xp(dev, torch.from_numpy(prevs).cuda(), d_state, N, 1, eos, temp, k, p)
    torch.cuda.synchronize()
    got = seq.cpu().numpy()[:, 0]
    gst = _state_from_dev(d_state)
    safe = dts > 1e-5
    assert (ln.cpu().numpy() == 1).all()
    assert (got[safe] == toks[safe]).all()
    # where the tokens agree the new interval and the code's place in it agree: the cells of the two
    # sides differ by rounding of the prefix sums only
    same = got == toks
    r_g, r_o = gst[same, 0].astype(np.float64), news[same, 0].astype(np.float64)
    np.testing.assert_allclose(r_g, r_o, rtol=1e-6)
    np.testing.assert_allclose(gst[same, 1].astype(np.float64) / r_g, news[same, 1].astype(np.float64) / r_o,
                               rtol=1e-6, atol=1e-9)
    return int(safe.sum()), len(toks), float((gst == news).all(axis=1).mean())


@pytest.mark.parametrize("dtype,V,ld,eos,temp,k,p", [
    (F32, 512, 512, 0, 1.0, 0, 1.0),          # rows in shared memory, fp64 exponential
    (BF16, 4096, 4096, 1, 0.8, 0, 1.0),       # ... masses from the bf16 table
    (BF16, 3001, 3001, -1, 0.9, 0, 1.0),      # rows off the 16-byte grid: general routine
    (F32, 1000, 1000, 7, 1.2, 0, 0.8),        # cuts: general routine
    (BF16, 2000, 2000, -1, 0.7, 20, 0.9),
    (BF16, 20000, 20000, 3, 0.8, 40, 1.0),
])
def test_steps_match_the_oracle_teacher_forced(B, orc, dtype, V, ld, eos, temp, k, p):
    rng = np.random.default_rng(V + k)
    rows = V if V <= 4096 else 64
    x = rng.normal(0, 2.5, (rows, ld)).astype(np.float32) - 1.5 * np.log(rng.permutation(ld) + 1.0)[None, :].astype(np.float32)
    if eos >= 0:
        x[:, eos] += 6.0
    table = _store(x, dtype)
    if rows < V:                                   # a tall table is not needed: tokens are folded into the rows there are
        full = np.zeros((V, ld), table.dtype)
        full[:rows] = table
        for r0 in range(rows, V, rows):
            full[r0:r0 + rows] = table[: min(rows, V - r0)]
        table = full
    dev = to_dev(table, dtype)
    N, S = 24, 2
    st0 = orc.xp_lattice_state(N, 0.377, S)
    prev0 = np.repeat(rng.integers(0, V, S), N).astype(np.int32)
    nsafe, nsteps, exact = _teacher_forced(B, orc, table, dtype, dev, prev0, st0, N, 10, eos, temp, k, p)
    assert nsafe > 0.9 * nsteps and nsteps >= 100
    assert exact > 0.98                            # nearly every step is bit for bit the oracle's


def test_long_decodes_equal_the_oracle_and_resume(B, orc):
    # whole sequences of 128 tokens on a c4-shaped table (cut to 4096 tokens): the GPU's free-running
    # decode equals the exact decoder's on nearly every lane (cells can differ by rounding, which a
    # code meets with probability ~1e-6 per step), dictionary order follows code order, all 128-token
    # sequences are distinct, and 128 steps = 50 + 78 from the returned state
    from paper_2210_15458_b200 import synth
    w = synth.c4(V=4096, S=8, T=128)
    table = w.table()
    dev = to_dev(table, BF16)
    u = w.shift()
    prev = np.repeat(w.starts(), w.N).astype(np.int32)
    st0 = orc.xp_lattice_state(w.N, u, w.S)
    ref = orc.xp_decode_bigram(table, BF16, prev, st0, w.N, w.T, -1, w.temp, threads=8)
    d_state = B.as_xp_lattice_state(w.N, u, 0, w.N, w.S)
    d_prev = torch.from_numpy(prev).cuda()
    status = torch.empty(w.lanes, dtype=torch.int32, device="cuda")
    seq, ln = B.as_decode_bigram_xp(dev, d_prev, d_state, w.N, w.T, -1, w.temp, lane_status=status)
    torch.cuda.synchronize()
    seq = seq.cpu().numpy()
    assert (status.cpu().numpy() == 0).all() and (ln.cpu().numpy() == w.T).all()
    same = (seq == ref.seq).all(axis=1)
    assert same.mean() >= 0.97
    assert np.array_equal(_state_from_dev(d_state)[same], ref.state[same])
    for s in range(w.S):
        grp = [tuple(r) for r in seq[s * w.N:(s + 1) * w.N]]
        assert grp == sorted(grp) and len(set(grp)) == w.N          # codes increase with j: so do the sequences
    # the fp64 code, for comparison, stops steering: its late tokens differ from the exact decode
    fp64 = orc.decode_bigram_codes(table, BF16, prev, np.tile(orc.lattice_codes(w.N, u), w.S), w.T, -1, w.temp, threads=8)
    assert (fp64.seq[:, :4] == ref.seq[:, :4]).all(axis=1).mean() > 0.95
    assert (fp64.seq[:, 64:] == ref.seq[:, 64:]).all(axis=1).mean() < 0.1
    # split and resume
    st_a = B.as_xp_lattice_state(w.N, u, 0, w.N, w.S)
    a_seq, _ = B.as_decode_bigram_xp(dev, d_prev, st_a, w.N, 50, -1, w.temp)
    b_seq, _ = B.as_decode_bigram_xp(dev, a_seq[:, 49].contiguous(), st_a, w.N, 78, -1, w.temp)
    torch.cuda.synchronize()
    assert np.array_equal(np.concatenate([a_seq.cpu().numpy(), b_seq.cpu().numpy()], axis=1), seq)
    assert torch.equal(st_a, d_state)


def test_whole_sequence_duplicates_follow_the_interval_width(B, orc):
    # Sec. 4.3 on whole sequences from the GPU: on a peaked model some 12-token sequences are wider than
    # 1/N and must repeat floor(N w) or ceil(N w) times; the GPU's multiplicities are those of the exact
    # decoder, whose own are pinned against exact interval widths on the CPU
    rng = np.random.default_rng(55)
    V, N, T = 8, 256, 12
    table = _store(rng.normal(0, 6.0, (V, V)), F32)
    for u in (0.0, 0.31, 0.999):
        st = B.as_xp_lattice_state(N, u)
        prev = torch.zeros(N, dtype=torch.int32, device="cuda")
        seq, _ = B.as_decode_bigram_xp(to_dev(table, F32), prev, st, N, T, -1)
        ref = orc.xp_decode_bigram(table, F32, np.zeros(N, np.int32), orc.xp_lattice_state(N, u), N, T, -1)
        seq = seq.cpu().numpy()
        assert (seq == ref.seq).all(axis=1).mean() > 0.99
        counts = {}
        for r in seq:
            counts[tuple(r)] = counts.get(tuple(r), 0) + 1
        assert max(counts.values()) > 1 and len(counts) > N // 8
        rows = [tuple(r) for r in seq]
        assert rows == sorted(rows)                          # equal sequences sit next to each other


def test_bad_state_and_bad_token_stop_the_lane(B):
    table = torch.zeros((16, 16), dtype=torch.float32, device="cuda")
    st = B.as_xp_lattice_state(4, 0.5)
    st[1, 0] = 5                                             # a range outside (2^62, 2^63]
    prev = torch.tensor([0, 0, 99, 0], dtype=torch.int32, device="cuda")
    status = torch.empty(4, dtype=torch.int32, device="cuda")
    seq, ln = B.as_decode_bigram_xp(table, prev, st, 4, 5, -1, lane_status=status)
    assert status.cpu().tolist() == [0, B.ERR_NUMERIC, B.ERR_NUMERIC, 0]
    assert ln.cpu().tolist() == [5, 0, 0, 5] and (seq[1].cpu().numpy() == -1).all()
