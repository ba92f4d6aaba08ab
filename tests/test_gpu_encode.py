"""Sequence -> interval on the GPU (the codebook of Sec. 4.1) against the CPU oracle.

Inputs to both sides are the oracle's own decoded sequences (or hand-made ones); the
round trip on the GPU's own output is checked as a property (the code lies inside the
interval of the sequence it decoded to), with no oracle value involved."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1
# per step the GPU's F and p differ from the oracle's by the rounding of an fp64 sum over
# at most V terms (relative <= V * 2^-53 ~ 4e-12 for V = 32128); T <= 128 steps compound.
RTOL_WIDTH = 1e-9
ATOL_LO = 1e-12


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


def gpu_encode(B, dev, prev, seq, ln, temp, k, p, V=None):
    st = torch.empty(len(prev), dtype=torch.int32, device="cuda")
    lo, wd = B.as_encode_bigram(dev, torch.from_numpy(prev).cuda(), torch.from_numpy(np.ascontiguousarray(seq)).cuda(),
                                torch.from_numpy(ln).cuda(), temp, k, p, V=V, lane_status=st)
    torch.cuda.synchronize()
    return lo.cpu().numpy(), wd.cpu().numpy(), st.cpu().numpy()


def compare(B, orc, table, dtype, dev, prev, seq, ln, temp, k, p, V=None):
    lo_r, wd_r, st_r = orc.encode_bigram(table, dtype, prev, seq, ln, temp, k, p, V=V)
    lo, wd, st = gpu_encode(B, dev, prev, seq, ln, temp, k, p, V=V)
    assert (st == st_r).all()
    np.testing.assert_allclose(wd, wd_r, rtol=RTOL_WIDTH, atol=0.0)
    np.testing.assert_allclose(lo, lo_r, rtol=RTOL_WIDTH, atol=ATOL_LO)
    return lo, wd, st


def test_encode_small_models_with_cuts_and_eos(B, orc):
    rng = np.random.default_rng(77)
    for dtype, V, eos, temp, k, p in [(F32, 50, 3, 1.0, 0, 1.0), (BF16, 300, 0, 0.8, 10, 1.0),
                                      (F32, 1000, 7, 1.2, 0, 0.8), (BF16, 2000, -1, 0.7, 20, 0.9),
                                      (F32, 4099, -1, 1.0, 1, 1.0), (BF16, 9001, 5, 0.9, 0, 1.0)]:
        x = rng.normal(0, 2, (V, V)).astype(np.float32)
        if eos >= 0:
            x[:, eos] += 3.0
        table = _store(x, dtype)
        dev = to_dev(table, dtype)
        prev = rng.integers(0, V, 64).astype(np.int32)
        codes = rng.random(64)
        ref = orc.decode_bigram_codes(table, dtype, prev, codes, 6, eos, temp, k, p, threads=8)
        seq, ln = ref.seq.astype(np.int32), ref.len.astype(np.int32)
        lo, wd, st = compare(B, orc, table, dtype, dev, prev, seq, ln, temp, k, p)
        assert (st == 0).all()
        # the oracle's sequences came from these codes: each code lies in its sequence's interval
        slack = 1e-9 * wd + 1e-15
        assert (lo <= codes + slack).all() and (codes < lo + wd + slack).all()


def test_encode_edge_cases(B, orc):
    rng = np.random.default_rng(5)
    V = 257
    x = rng.normal(0, 2, (V, V)).astype(np.float32)
    x[4, 9] = -np.inf                                      # masked token
    table = _store(x, F32)
    dev = to_dev(table, F32)
    order = np.argsort(-x[0], kind="stable")
    prev = np.array([0, 0, 0, 0, 4, 0, 0], np.int32)
    seq = np.full((7, 5), -1, np.int32)
    ln = np.zeros(7, np.int32)
    seq[0, :3] = [order[0], 2, 3]; ln[0] = 3              # fine under top-k only if 2, 3 survive: checked vs oracle
    ln[1] = 0                                             # empty sequence: [0, 1)
    seq[2, :2] = [order[0], order[0]]; ln[2] = 9          # length above T is read as T
    seq[2, 2:] = order[0]
    seq[3, :2] = [order[0], V + 3]; ln[3] = 2             # token id out of range
    seq[4, :1] = [9]; ln[4] = 1                           # masked token
    seq[5, :2] = [order[V - 1], 1]; ln[5] = 2             # cut by top-k at the first step
    seq[6, :1] = [order[2]]; ln[6] = 1
    for temp, k, p in [(1.0, 0, 1.0), (0.9, 3, 1.0), (1.0, 0, 0.3)]:
        lo, wd, st = compare(B, orc, table, F32, dev, prev, seq, ln, temp, k, p)
        assert st[1] == 0 and lo[1] == 0.0 and wd[1] == 1.0
        assert st[3] == B.ERR_INVALID_ARG and st[4] == B.ERR_NUMERIC
        if k:
            assert st[5] == B.ERR_NUMERIC and lo[5] == 0.0 and wd[5] == 1.0
    # lanes = 0 and T = 0
    lo, wd = B.as_encode_bigram(dev, torch.empty(0, dtype=torch.int32, device="cuda"),
                                torch.empty((0, 4), dtype=torch.int32, device="cuda"),
                                torch.empty(0, dtype=torch.int32, device="cuda"))
    assert lo.numel() == 0
    lo, wd = B.as_encode_bigram(dev, torch.zeros(2, dtype=torch.int32, device="cuda"),
                                torch.empty((2, 0), dtype=torch.int32, device="cuda"),
                                torch.full((2,), 3, dtype=torch.int32, device="cuda"))
    assert lo.cpu().tolist() == [0.0, 0.0] and wd.cpu().tolist() == [1.0, 1.0]


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_encode_one_token_sequences_tile_the_unit_interval(B, orc, dtype):
    # every one-token sequence of a row: the intervals are adjacent, in index order, and cover [0,1)
    rng = np.random.default_rng(8)
    V = 3001
    x = rng.normal(0, 3, (4, V)).astype(np.float32)
    x[1, ::7] = -np.inf
    x[2] = np.round(x[2])                                  # many ties
    table = np.zeros((V, V + 3), np.float32)               # padded leading dimension
    table[:4, :V] = x
    table = _store(table, dtype)
    dev = to_dev(table, dtype)
    for row, (temp, k, p) in [(0, (1.0, 0, 1.0)), (1, (0.7, 0, 1.0)), (2, (1.0, 40, 1.0)), (2, (1.0, 0, 0.7)),
                              (3, (1.5, 100, 0.9))]:
        prev = np.full(V, row, np.int32)
        seq = np.arange(V, dtype=np.int32)[:, None].copy()
        ln = np.ones(V, np.int32)
        lo, wd, st = compare(B, orc, table, dtype, dev, prev, seq, ln, temp, k, p, V=V)
        ok = st == 0
        assert ok.sum() >= 1 and ((st == 0) | (st == B.ERR_NUMERIC)).all()
        assert abs(wd[ok].sum() - 1.0) < 1e-12
        np.testing.assert_allclose(lo[ok][1:], (lo[ok] + wd[ok])[:-1], rtol=0, atol=1e-13)
        assert lo[ok][0] == 0.0
        if k:
            assert ok.sum() == k or p < 1.0


def test_encode_c1_and_round_trip_of_the_gpu_decode(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c1()
    table = w.table()
    dev = to_dev(table, F32)
    starts = w.starts()
    u = w.shift()
    prev = np.repeat(starts, w.N).astype(np.int32)
    codes = np.tile(orc.lattice_codes(w.N, u), w.S)
    ref = orc.decode_bigram_codes(table, F32, prev, codes, w.T, w.eos, w.temp, 0, 1.0, threads=8)
    compare(B, orc, table, F32, dev, prev, ref.seq.astype(np.int32), ref.len.astype(np.int32), w.temp, 0, 1.0)
    # property on the GPU's own decode: the first steps' interval holds the code that produced them
    Tshort = 4
    seq, ln = B.as_decode_bigram(dev, torch.from_numpy(starts).cuda(), w.N, u, Tshort, w.eos, w.temp)
    lo, wd = B.as_encode_bigram(dev, torch.from_numpy(prev).cuda(), seq, ln, w.temp)
    torch.cuda.synchronize()
    lo, wd = lo.cpu().numpy(), wd.cpu().numpy()
    slack = 1e-9 * wd + 1e-15
    assert (lo <= codes + slack).all() and (codes < lo + wd + slack).all()
    # Sec. 4.3: within a group the lattice spacing 1/N bounds how many lanes share one sequence
    assert (wd > 0).all()


def test_encode_c4_full_size_sampled(B, orc):
    from paper_2210_15458_b200 import synth
    w = synth.c4()
    table = w.table()
    dev = to_dev(table, BF16)
    lanes = np.sort(np.random.default_rng(4).choice(w.lanes, 24, replace=False))
    prev = np.repeat(w.starts(), w.N).astype(np.int32)[lanes]
    codes = np.tile(orc.lattice_codes(w.N, w.shift()), w.S)[lanes]
    ref = orc.decode_bigram_codes(table, BF16, prev, codes, 24, w.eos, w.temp, 0, 1.0, threads=8)
    lo, wd, st = compare(B, orc, table, BF16, dev, prev, ref.seq.astype(np.int32), ref.len.astype(np.int32),
                         w.temp, 0, 1.0)
    assert (st == 0).all()
