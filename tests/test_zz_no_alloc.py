"""as_step_host_static: the host-buffer step for callers that may not allocate device memory.

Some users of this library get a stream from a host application but no right to device memory
(the application keeps the GPU in its own pool), or sit on a path where a cudaMalloc would stall
every stream of the device.  For them the library carries its own work buffer.  This test calls
that entry point through the C ABI twice in a row (the buffer keeps the first call's contents,
the second call must not be disturbed by them) and compares with as_step_host, which uses a
caller-supplied buffer -- the same kernel on the same bytes, so the results must be equal bit
for bit; it checks that the device's free memory is the same before and after the calls, and
that an oversized request is refused.  It is collected
last so that a run stopping at the first failure has already run everything else."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_15458_b200 import binding
    binding.lib()
    return binding


def _host_inputs(lanes, V, seed):
    from paper_2210_15458_b200 import synth
    rng = np.random.default_rng(seed)
    bits = synth.f32_to_bf16_bits(rng.normal(0, 3, (lanes, V)).astype(np.float32))
    logits = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    codes = torch.from_numpy(rng.random(lanes))
    return logits, codes


def test_static_work_buffer_matches_caller_buffer_twice(B):
    cases = [(200, 32000, 0.7, 40, 1.0), (64, 9001, 1.1, 0, 0.9)]
    inputs, wanted = [], []
    for call, (lanes, V, temp, k, p) in enumerate(cases):
        logits, codes = _host_inputs(lanes, V, 40 + call)
        tok = torch.empty(lanes, dtype=torch.int32)
        c = torch.empty(lanes, dtype=torch.float64)
        st = torch.empty(lanes, dtype=torch.int32)
        work = torch.empty(B.as_step_host_work_bytes(B.BF16, lanes, V) + 256, dtype=torch.uint8, device="cuda")
        B.as_step_host(logits, codes, temp, k, p, tok, c, st, work)
        inputs.append((logits, codes))
        wanted.append((tok, c, st))
    # a first call on this device (it looks up the buffer's address), then the measured ones
    lanes, V, temp, k, p = cases[0]
    warm = (torch.empty(lanes, dtype=torch.int32), torch.empty(lanes, dtype=torch.float64))
    B.as_step_host_static(inputs[0][0], inputs[0][1], temp, k, p, warm[0], warm[1], None)
    outs = [(torch.full((c[0],), -7, dtype=torch.int32), torch.full((c[0],), -7.0, dtype=torch.float64),
             torch.full((c[0],), -7, dtype=torch.int32)) for c in cases]
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    # two calls in a row on the built-in buffer: the second finds the first one's bytes in it
    for (lanes, V, temp, k, p), (logits, codes), (got_tok, got_c, got_st) in zip(cases, inputs, outs):
        B.as_step_host_static(logits, codes, temp, k, p, got_tok, got_c, got_st)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "as_step_host_static changed the device's free memory"
    for (got_tok, got_c, got_st), (want_tok, want_c, want_st) in zip(outs, wanted):
        assert (got_st == 0).all() and torch.equal(got_st, want_st)
        assert torch.equal(got_tok, want_tok)
        assert torch.equal(got_c, want_c)                  # same kernel, same bytes: bit for bit


def test_static_work_buffer_refuses_what_does_not_fit(B):
    lanes, V = 600, 32000                       # 38 MB of bf16 logits > the 24 MiB buffer
    assert B.as_step_host_work_bytes(B.BF16, lanes, V) > B.STATIC_WORK_BYTES
    logits, codes = _host_inputs(lanes, V, 3)
    tok = torch.empty(lanes, dtype=torch.int32)
    out = torch.empty(lanes, dtype=torch.float64)
    with pytest.raises(B.AsError) as e:
        B.as_step_host_static(logits, codes, 1.0, 0, 1.0, tok, out, None)
    assert e.value.code == B.ERR_UNSUPPORTED and "AS_STATIC_WORK_BYTES" in str(e.value)
