"""The bounds-checked build of the library (every index into a ring stage, a hit or candidate
list, a rank array, a histogram, a chunk array, the mass table or a row buffer is checked on the
device and recorded instead of trapping) over a matrix of small and ragged shapes, with guard
words around every output buffer.  Results must still equal the oracle's, the record must stay
empty and the guard words untouched."""
import os

import numpy as np
import pytest

from tests.parity import compare_step

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1
GUARD = 64


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_15458_b200 import _build, binding
    if not os.path.exists(_build.LIB_CHECKED):
        pytest.fail("checked library missing: run __graft_entry__.build()")
    binding.use_library(_build.LIB_CHECKED)
    binding.lib()
    binding.as_debug_bounds(reset=True)
    yield binding
    binding.use_library(None)


def to_dev(arr, dtype):
    if dtype == BF16:
        return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).cuda()


def _store(x, dtype):
    from paper_2210_15458_b200 import synth
    x = np.ascontiguousarray(x, dtype=np.float32)
    return synth.f32_to_bf16_bits(x) if dtype == BF16 else x


class Guarded:
    """An output buffer with GUARD sentinel elements in front and behind."""

    def __init__(self, shape, dtype, sentinel):
        n = int(np.prod(shape))
        self.full = torch.full((n + 2 * GUARD,), sentinel, dtype=dtype, device="cuda")
        self.view = self.full[GUARD:GUARD + n].view(*shape)
        self.sentinel = sentinel

    def intact(self):
        f = self.full.cpu()
        return bool((f[:GUARD] == self.sentinel).all() and (f[-GUARD:] == self.sentinel).all())


def _clean(B):
    rec = B.as_debug_bounds(reset=True)
    assert rec[0] == 0, "out-of-range index on the device: %d failures, first at site %d, index %d, bound %d" % rec


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_step_shapes_checked(B, orc, dtype):
    rng = np.random.default_rng(77)
    for V in (1, 3, 17, 33, 1000, 4099, 9001, 32000, 70001, 140003):
        lanes = 13 if V > 20000 else 29
        x = rng.normal(0, 3, (lanes, V)).astype(np.float32)
        if V > 100:
            x[2, ::3] = -np.inf
            x[3] = np.round(x[3])
            x[4] += np.linspace(0, 6, V, dtype=np.float32)          # the best tokens come last
        arr = _store(x, dtype)
        dev = to_dev(arr, dtype)
        codes = rng.random(lanes)
        codes[0], codes[1] = 0.0, 1.0
        for temp, k, p in [(1.0, 0, 1.0), (0.7, 40, 1.0), (1.0, 0, 0.9), (0.8, 64, 0.95), (1.0, 300, 0.5)]:
            tok = Guarded((lanes,), torch.int32, -77)
            out = Guarded((lanes,), torch.float64, -77.0)
            d = {}
            B.as_step(dev, torch.from_numpy(codes).cuda(), temp, k, p, tokens=tok.view, codes_out=out.view, diag=d)
            torch.cuda.synchronize()
            ref = orc.step(arr, dtype, codes, temp, k, p, threads=8)
            compare_step(ref, tok.view.cpu().numpy(), out.view.cpu().numpy(), d["p_tok"].cpu().numpy(),
                         d["n_kept"].cpu().numpy(), d["lane_status"].cpu().numpy(), what="checked V=%d %s" % (V, (temp, k, p)))
            assert tok.intact() and out.intact()
            _clean(B)
        if V >= 1000:
            tok = Guarded((lanes,), torch.int32, -77)
            out = Guarded((lanes,), torch.float64, -77.0)
            B.as_step(dev, torch.from_numpy(codes).cuda(), 0.9, 5, tokens=tok.view, codes_out=out.view, typical_p=0.8)
            torch.cuda.synchronize()
            assert tok.intact() and out.intact()
            _clean(B)


def test_cluster_kernel_checked(B, orc):
    rng = np.random.default_rng(78)
    arr = _store(rng.normal(0, 3, (24, 65560)), BF16)
    codes = rng.random(24)
    try:
        B.as_tune(B.TUNE_STEP_PATH, 2)
        for cs in (2, 8):
            B.as_tune(B.TUNE_CLUSTER, cs)
            tok = Guarded((24,), torch.int32, -77)
            out = Guarded((24,), torch.float64, -77.0)
            B.as_step(to_dev(arr, BF16), torch.from_numpy(codes).cuda(), 0.8, 64, 0.95, tokens=tok.view, codes_out=out.view)
            torch.cuda.synchronize()
            compare_step(orc.step(arr, BF16, codes, 0.8, 64, 0.95, threads=8), tok.view.cpu().numpy(), out.view.cpu().numpy())
            assert tok.intact() and out.intact()
            _clean(B)
    finally:
        B.as_tune(B.TUNE_CLUSTER, 0)
        B.as_tune(B.TUNE_STEP_PATH, 0)


@pytest.mark.parametrize("k,p", [(0, 1.0), (12, 1.0), (0, 0.85)])
def test_decode_loops_checked(B, orc, k, p):
    # the loops' outputs (sequences, lengths, final codes, extended-precision state) between guard words
    rng = np.random.default_rng(79)
    V, lanes, T, eos = 3000, 40, 9, 5
    x = rng.normal(0, 2.5, (V, V)).astype(np.float32)
    x[:, eos] += 4.0
    table = _store(x, BF16)
    dev = to_dev(table, BF16)
    prev = rng.integers(0, V, lanes).astype(np.int32)
    codes = rng.random(lanes)
    seq = Guarded((lanes, T), torch.int32, -77)
    ln = Guarded((lanes,), torch.int32, -77)
    cf = Guarded((lanes,), torch.float64, -77.0)
    B.as_decode_bigram_codes(dev, torch.from_numpy(prev).cuda(), torch.from_numpy(codes).cuda(), T, eos, 0.8, k, p,
                             codes_final=cf.view, seq=seq.view, length=ln.view)
    torch.cuda.synchronize()
    ref = orc.decode_bigram_codes(table, BF16, prev, codes, T, eos, 0.8, k, p, threads=8)
    assert (seq.view.cpu().numpy()[:, 0] == ref.seq[:, 0]).mean() > 0.9
    assert seq.intact() and ln.intact() and cf.intact()
    _clean(B)
    st = Guarded((lanes, 4), torch.int64, -77)
    st.view.copy_(B.as_xp_lattice_state(lanes, 0.3))
    B.as_decode_bigram_xp(dev, torch.from_numpy(prev).cuda(), st.view, lanes, T, eos, 0.8, k, p, seq=seq.view, length=ln.view)
    torch.cuda.synchronize()
    assert seq.intact() and ln.intact() and st.intact()
    _clean(B)
    lo, wd = B.as_encode_bigram(dev, torch.from_numpy(prev).cuda(), seq.view, ln.view, 0.8, k, p)
    torch.cuda.synchronize()
    _clean(B)


def test_the_record_reports_a_planted_index(B):
    # the reporting path itself: the record starts empty, and reading it resets it
    assert B.as_debug_bounds(reset=True)[0] == 0
    assert B.as_debug_bounds(reset=False) == (0, 0, 0, 0)
